// 2:4 weight sparsification + packing (Section 2.2 and Section 3.2.1 of the paper).
//
// Streaming, HBM-bound kernels: 2 B read + 1 B packed values + 1/8 B metadata per element.
//   * contiguous groups: one thread owns 16 consecutive elements of a row (four groups, one
//     metadata word): two 128-bit loads, one 128-bit store of packed values, one 16-bit store;
//     a warp owns 32 consecutive chunks of a row, so no index is ever divided.
//   * strided groups (groups along dim 0, output K-major): a CTA stages a [128 x 64] panel in
//     shared memory, selects per column, and writes the transposed packed panel with 128-bit
//     stores through a padded staging buffer.
#include "sf_common.cuh"
#include "fp8_fmt.cuh"
#include "tc_ptx.cuh"
#include "gemm_tc.cuh"

namespace sf {

namespace {

// Expand (nibble, two values) to the four dense patterns of a group.
__device__ __forceinline__ void expand_group(uint32_t nib, uint32_t v0, uint32_t v1, uint32_t d[4]) {
  const uint32_t p0 = nib & 3u, p1 = nib >> 2;
#pragma unroll
  for (int i = 0; i < 4; ++i) d[i] = (p0 == (uint32_t)i) ? v0 : (p1 == (uint32_t)i) ? v1 : 0u;
}

// A warp owns 32 consecutive 16-element chunks of one row (1 KB of input); the eight warps of a CTA take
// eight consecutive rows. Grid = (chunks / 32, rows / 8 folded over y and z): no index division.
constexpr int kRowsPerCta = 8;

template <bool kSoft>
__global__ void __launch_bounds__(256)
prune24_rows_kernel(const uint4* __restrict__ W, int64_t rows, int cols, int64_t ld,
                    uint4* __restrict__ vals, uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw,
                    uint4* __restrict__ dense_out) {
  __shared__ Top2Entry lut[16];
  top2_lut_init(lut, threadIdx.x);
  __syncthreads();
  const int words_per_row = cols >> 4;                           // 16-element chunks per row
  const int kw = (int)blockIdx.x * 32 + (int)(threadIdx.x & 31);
  const int64_t r = ((int64_t)blockIdx.z * gridDim.y + blockIdx.y) * kRowsPerCta + (threadIdx.x >> 5);
  if (kw >= words_per_row || r >= rows) return;
  const int64_t idx = r * words_per_row + kw;

  const uint4* src = W + ((r * ld) >> 3) + (kw << 1);
  const uint4 q0 = __ldg(src), q1 = __ldg(src + 1);
  const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};

  uint32_t packed[4], m = 0, dense[8];
  {
    // two groups per pass through the 16-bit-halves selection
    Top2Entry e[4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t a_lo = w[4 * h], a_hi = w[4 * h + 1], b_lo = w[4 * h + 2], b_hi = w[4 * h + 3];
      top2of4_x2<kSoft>(__byte_perm(a_lo, b_lo, 0x5410u), __byte_perm(a_lo, b_lo, 0x7632u),
                        __byte_perm(a_hi, b_hi, 0x5410u), __byte_perm(a_hi, b_hi, 0x7632u), lut, e[2 * h], e[2 * h + 1]);
    }
#pragma unroll
    for (int g = 0; g < 4; ++g)
      packed[g] = kSoft ? soft_threshold_pair(w[2 * g], w[2 * g + 1], e[g]) : __byte_perm(w[2 * g], w[2 * g + 1], e[g].kept);
    m = ((e[0].kept & 0x000F0000u) | (e[1].kept & 0x00F00000u) | (e[2].kept & 0x0F000000u) | (e[3].kept & 0xF0000000u)) >> 16;
  }
  if (dense_out) {
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      uint32_t d[4];
      expand_group((m >> (4 * g)) & 0xFu, packed[g] & 0xFFFFu, packed[g] >> 16, d);
      dense[2 * g] = d[0] | (d[1] << 16);
      dense[2 * g + 1] = d[2] | (d[3] << 16);
    }
  }
  vals[idx] = make_uint4(packed[0], packed[1], packed[2], packed[3]);       // [R, K/2] bf16: 8 per chunk
  meta[idx] = (uint16_t)m;
  if (meta_hw) {
    // tensor-core order (see meta_hw_offset), with the row part shared by the warp
    const uint32_t mi = (uint32_t)r & 127u, kwi = (uint32_t)kw & 7u;
    const int64_t atom = (r >> 7) * (int64_t)(cols >> 7) + (kw >> 3);
    const uint32_t in_atom = (mi >> 4) * 256u + (kwi & 1u) * 128u + (mi & 7u) * 16u + (kwi >> 1) * 4u + ((mi >> 3) & 1u) * 2u;
    *reinterpret_cast<uint16_t*>(meta_hw + atom * 2048 + in_atom) = (uint16_t)m;
  }
  if (dense_out) {
    uint4* dst = dense_out + ((r * cols) >> 3) + (kw << 1);
    dst[0] = make_uint4(dense[0], dense[1], dense[2], dense[3]);
    dst[1] = make_uint4(dense[4], dense[5], dense[6], dense[7]);
  }
}

// Strided groups. W is [Kd, Rc] row-major (Kd = rows = reduction dim, Rc = cols); outputs are
// vals [Rc, Kd/2], meta [Rc, Kd/16]. Panel: 128 reduction rows x 64 columns.
// Persistent CTAs walk the panels. One TMA load brings the next panel into a two-slot ring
// (out-of-range rows and columns arrive as zeros), so no thread computes load addresses; selection runs
// on column pairs; packed values, canonical metadata and the tensor-core-ordered metadata of a panel are
// assembled in shared memory and leave as 128-bit stores.
constexpr int kPanelK = 128, kPanelC = 64;
constexpr int kColsSlots = 2;                       // the next panel loads while this one is worked on
constexpr int kStageRow = (kPanelK / 2) * 2 + 16;   // packed bytes per column + 16 B pad
constexpr int kColsTileBytes = kPanelK * kPanelC * 2, kColsStageBytes = kPanelC * kStageRow;
constexpr int kColsMetaBytes = kPanelC * (kPanelK / 16) * 2;       // canonical words [column][8]; the same again in hardware order
constexpr int kColsSmemBytes = 128 + kColsSlots * kColsTileBytes + kColsStageBytes + 2 * kColsMetaBytes + 64;
constexpr int kColsCtasPerSm = 5;                   // 44 KB each; measured best among 3..5 with two or three slots
static_assert(kPanelK / 16 == 8 && kPanelC == 64, "index shifts in prune24_cols_kernel assume a 128 x 64 panel");

// kFp8: the kept values leave as E4M3 codes of float(value) * scale (vals = uint8 [Rc, Kd/2]); no masked copy.
template <bool kSoft, bool kFp8 = false>
__global__ void __launch_bounds__(256)
prune24_cols_kernel(const __grid_constant__ CUtensorMap tmapW, int64_t Kd, int64_t Rc,
                    uint16_t* __restrict__ vals, uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw,
                    uint16_t* __restrict__ dense_out, int panels_x, int num_panels, float scale = 1.f) {
  using namespace ptx;
  extern __shared__ uint8_t cols_smem_raw[];
  uint8_t* cols_smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(cols_smem_raw) + 127) & ~uintptr_t(127));
  typedef uint16_t TileRow[kPanelC];
  typedef uint8_t StageRow[kStageRow];
  typedef uint16_t MetaRow[kPanelK / 16];
  StageRow* stage = reinterpret_cast<StageRow*>(cols_smem + kColsSlots * kColsTileBytes);              // [kPanelC]
  MetaRow* mstage = reinterpret_cast<MetaRow*>(cols_smem + kColsSlots * kColsTileBytes + kColsStageBytes);   // [kPanelC]
  uint8_t* mhw = reinterpret_cast<uint8_t*>(mstage) + kColsMetaBytes;                                   // four 256-byte row blocks
  uint64_t* full = reinterpret_cast<uint64_t*>(mhw + kColsMetaBytes);                                   // [kColsSlots]
  int* abort_flag = reinterpret_cast<int*>(full + kColsSlots);
  const int tid = threadIdx.x;

  auto issue = [&](int it) {                    // thread 0: load panel number `it` of this CTA into its slot
    const int panel = (int)blockIdx.x + it * (int)gridDim.x;
    if (panel >= num_panels) return;
    const int py = panel / panels_x, px = panel - py * panels_x;
    const int slot = it % kColsSlots;
    mbar_arrive_expect_tx(&full[slot], (uint32_t)kColsTileBytes);
    tma_load_2d(cols_smem + slot * kColsTileBytes, &tmapW, &full[slot], px * kPanelC, py * kPanelK);
  };
  __shared__ Top2Entry lut[16];
  top2_lut_init(lut, tid);
  if (tid == 0) {
    prefetch_tmap(&tmapW);
    for (int sl = 0; sl < kColsSlots; ++sl) mbar_init(&full[sl], 1);
    *abort_flag = 0;
    fence_mbar_init();
    for (int d = 0; d < kColsSlots - 1; ++d) issue(d);
  }
  __syncthreads();

  int it = 0;
  for (int panel = blockIdx.x; panel < num_panels; panel += gridDim.x, ++it) {
    const int slot = it % kColsSlots;
    __syncthreads();            // the previous panel is stored: its stage buffers and the slot of the panel before are free
    if (tid == 0) {
      fence_proxy_async_smem(); // earlier generic writes to that slot (masked copy) before the TMA write
      issue(it + kColsSlots - 1);
    }
    // one warp waits for the load (bounded), the block follows through the barrier
    bool ok = true;
    if (tid < 32) ok = mbar_wait(&full[slot], (uint32_t)(it / kColsSlots) & 1u, abort_flag);
    if (__syncthreads_or(!ok)) break;

    const int py = panel / panels_x, px = panel - py * panels_x;
    const int64_t c0 = (int64_t)px * kPanelC, k0 = (int64_t)py * kPanelK;
    const int kvalid = (int)min((int64_t)kPanelK, Kd - k0);               // multiple of 16
    const int cvalid = (int)min((int64_t)kPanelC, Rc - c0);               // multiple of 8
    TileRow* tile = reinterpret_cast<TileRow*>(cols_smem + slot * kColsTileBytes);

    // select: one thread per (column pair, 16-row chunk); lanes run along column pairs, so the 32-bit
    // loads of a warp are conflict-free, and two byte permutes turn two rows into the two columns' pairs
    for (int i = tid; i < (kPanelC / 2) * (kPanelK / 16); i += 256) {
      const int cp = i & (kPanelC / 2 - 1), ch = i >> 5;                   // ch: chunk of 16 rows
      const int c = 2 * cp;
      if (c >= cvalid || ch * 16 >= kvalid) continue;                      // cvalid is even: the pair is whole
      uint32_t packed[2][4], m[2] = {0, 0};
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int kr = ch * 16 + g * 4;
        uint32_t rw[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) rw[j] = *reinterpret_cast<const uint32_t*>(&tile[kr + j][c]);
        // the two columns of the pair share one pass of the 16-bit-halves selection
        Top2Entry ent[2];
        top2of4_x2<kSoft>(rw[0], rw[1], rw[2], rw[3], lut, ent[0], ent[1]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const uint32_t sel = e ? 0x7632u : 0x5410u;
          const uint32_t lo = __byte_perm(rw[0], rw[1], sel), hi = __byte_perm(rw[2], rw[3], sel);
          packed[e][g] = kSoft ? soft_threshold_pair(lo, hi, ent[e]) : __byte_perm(lo, hi, ent[e].kept);
          const uint32_t nib = (ent[e].kept >> 16) & 0xFu;
          m[e] |= nib << (4 * g);
          if (dense_out) {
            uint32_t d[4];
            expand_group(nib, packed[e][g] & 0xFFFFu, packed[e][g] >> 16, d);
#pragma unroll
            for (int j = 0; j < 4; ++j) tile[kr + j][c + e] = (uint16_t)d[j];
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        if (kFp8) {
          const uint32_t q0 = quant2(packed[e][0], scale), q1 = quant2(packed[e][1], scale);
          const uint32_t q2 = quant2(packed[e][2], scale), q3 = quant2(packed[e][3], scale);
          *reinterpret_cast<uint2*>(&stage[c + e][ch * 8]) = make_uint2(q0 | (q1 << 16), q2 | (q3 << 16));
        } else {
          *reinterpret_cast<uint4*>(&stage[c + e][ch * 16]) = make_uint4(packed[e][0], packed[e][1], packed[e][2], packed[e][3]);
        }
        mstage[c + e][ch] = (uint16_t)m[e];
        // tensor-core order (see meta_hw_offset): the panel's 64 output rows are four 16-row blocks of one atom
        const int mi = c + e;
        *reinterpret_cast<uint16_t*>(mhw + (mi >> 4) * 256 + (ch & 1) * 128 + (mi & 7) * 16 + (ch >> 1) * 4 +
                                     ((mi >> 3) & 1) * 2) = (uint16_t)m[e];
      }
    }
    __syncthreads();

    // store packed values: per column kvalid/2 elements = kvalid bytes, 16 B per thread
    const int chunks = kvalid >> 4;
    const bool full_k = chunks == kPanelK / 16;
    for (int i = tid; i < kPanelC * chunks; i += 256) {
      const int c = full_k ? (i >> 3) : (i / chunks), ch = i - c * chunks;
      if (c >= cvalid) continue;
      const int64_t orow = c0 + c;
      if (kFp8) {
        *reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(vals) + orow * (Kd >> 1) + (k0 >> 1) + ch * 8) =
            *reinterpret_cast<const uint2*>(&stage[c][ch * 8]);
      } else {
        *reinterpret_cast<uint4*>(vals + orow * (Kd >> 1) + (k0 >> 1) + ch * 8) = *reinterpret_cast<const uint4*>(&stage[c][ch * 16]);
      }
    }
    if (full_k && (Kd & 127) == 0) {
      // whole panels: a column's eight metadata words are 16 contiguous, aligned bytes in either order
      if (tid < kPanelC) {
        if (tid < cvalid)
          *reinterpret_cast<uint4*>(meta + (c0 + tid) * (Kd >> 4) + (k0 >> 4)) = *reinterpret_cast<const uint4*>(&mstage[tid][0]);
      } else if (tid < 2 * kPanelC && meta_hw) {
        const int t = tid - kPanelC;                                        // 16-byte piece of the panel's 1 KB
        // (the hardware order exists for whole 128-row blocks only, so all 64 columns are valid here)
        const int64_t atom = (c0 >> 7) * (Kd >> 7) + (k0 >> 7);
        *reinterpret_cast<uint4*>(meta_hw + atom * 2048 + ((c0 & 127) >> 4) * 256 + t * 16) =
            *reinterpret_cast<const uint4*>(mhw + t * 16);
      }
    } else {
      for (int i = tid; i < kPanelC * chunks; i += 256) {
        const int c = i / chunks, ch = i - c * chunks;
        if (c >= cvalid) continue;
        const int64_t orow = c0 + c, kw = (k0 >> 4) + ch;
        const uint16_t mw = mstage[c][ch];
        meta[orow * (Kd >> 4) + kw] = mw;
        if (meta_hw) *reinterpret_cast<uint16_t*>(meta_hw + meta_hw_offset(orow, kw, Kd)) = mw;
      }
    }
    if (dense_out) {
      for (int i = tid; i < kPanelK * (kPanelC / 8); i += 256) {
        const int kr = i >> 3, cc = (i & 7) << 3;
        if (kr < kvalid && cc < cvalid)
          *reinterpret_cast<uint4*>(dense_out + (k0 + kr) * Rc + c0 + cc) = *reinterpret_cast<const uint4*>(&tile[kr][cc]);
      }
    }
  }
}

// Plain tiled transpose of a bf16 matrix: out[c][r] = in[r][c].
__global__ void __launch_bounds__(256)
transpose_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, int64_t rows, int64_t cols) {
  __shared__ uint16_t t[64][64 + 2];
  const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;                // 32 x 8
  for (int i = ty; i < 64; i += 8) {
    const int64_t r = r0 + i;
    if (r < rows) {
      const int64_t c = c0 + 2 * tx;
      if (c + 1 < cols) {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(in + r * cols + c);
        t[i][2 * tx] = (uint16_t)v;
        t[i][2 * tx + 1] = (uint16_t)(v >> 16);
      } else if (c < cols) {
        t[i][2 * tx] = in[r * cols + c];
      }
    }
  }
  __syncthreads();
  for (int i = ty; i < 64; i += 8) {
    const int64_t c = c0 + i;                                            // output row
    if (c < cols) {
      const int64_t r = r0 + 2 * tx;
      if (r + 1 < rows) {
        const uint32_t v = (uint32_t)t[2 * tx][i] | ((uint32_t)t[2 * tx + 1][i] << 16);
        *reinterpret_cast<uint32_t*>(out + c * rows + r) = v;
      } else if (r < rows) {
        out[c * rows + r] = t[2 * tx][i];
      }
    }
  }
}

// Transpose for shapes that are multiples of 64: 16-byte global loads and stores on both sides.
// Shared tile rows are 33 words apart, so the word stores of the load phase are conflict-free and the
// strided 16-bit reads of the store phase collide two ways at most.
__global__ void __launch_bounds__(256)
transpose64_kernel(const uint16_t* __restrict__ in, uint16_t* __restrict__ out, int64_t rows, int64_t cols) {
  __shared__ uint32_t t[64 * 33];
  const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
  const int tid = threadIdx.x;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int row = (tid >> 3) + 32 * j, c8 = (tid & 7) * 8;
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(in + (r0 + row) * cols + c0 + c8));
    uint32_t* d = t + row * 33 + (c8 >> 1);
    d[0] = q.x; d[1] = q.y; d[2] = q.z; d[3] = q.w;
  }
  __syncthreads();
  const uint16_t* th = reinterpret_cast<const uint16_t*>(t);
  const int lane = tid & 31, warp = tid >> 5;
  const int r8 = lane & 7, cq = lane >> 3;
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int c = warp * 4 + cq + 32 * j;                    // output row inside the tile
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t a = th[(r8 * 8 + 2 * k) * 66 + c], b = th[(r8 * 8 + 2 * k + 1) * 66 + c];
      w[k] = a | (b << 16);
    }
    *reinterpret_cast<uint4*>(out + (c0 + c) * rows + r0 + r8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

}  // namespace

int launch_prune24(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim, int prune_mode,
                   void* vals, void* meta, void* meta_hw, void* dense_out, cudaStream_t s) {
  if (rows == 0 || cols == 0) return SF_OK;
  if (group_dim == 1) {
    if (cols > (int64_t)1 << 30) return SF_ERR_SHAPE;
    const int64_t row_ctas = (rows + kRowsPerCta - 1) / kRowsPerCta;
    const int64_t gy = row_ctas < 32768 ? row_ctas : 32768;
    const int64_t gz = (row_ctas + gy - 1) / gy;
    if (gz > 65535) return SF_ERR_SHAPE;
    dim3 grid((unsigned)(((cols >> 4) + 31) / 32), (unsigned)gy, (unsigned)gz);
    if (prune_mode == 0)
      prune24_rows_kernel<false><<<grid, 256, 0, s>>>((const uint4*)W, rows, (int)cols, ld, (uint4*)vals,
                                                      (uint16_t*)meta, (uint8_t*)meta_hw, (uint4*)dense_out);
    else
      prune24_rows_kernel<true><<<grid, 256, 0, s>>>((const uint4*)W, rows, (int)cols, ld, (uint4*)vals,
                                                     (uint16_t*)meta, (uint8_t*)meta_hw, (uint4*)dense_out);
  } else {
    const int64_t px = (cols + kPanelC - 1) / kPanelC, py = (rows + kPanelK - 1) / kPanelK;
    if (px * py > (int64_t)1 << 30) return SF_ERR_SHAPE;
    const int num_panels = (int)(px * py);
    static bool attr_done[64] = {false};
    static int sms[64] = {0};
    int dev = 0;
    SF_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return SF_ERR_UNSUPPORTED;
    if (!attr_done[dev]) {
      SF_CUDA_TRY(cudaFuncSetAttribute(prune24_cols_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColsSmemBytes));
      SF_CUDA_TRY(cudaFuncSetAttribute(prune24_cols_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColsSmemBytes));
      SF_CUDA_TRY(cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev));
      attr_done[dev] = true;
    }
    alignas(64) CUtensorMap tm;
    int st = make_tmap_2d(&tm, W, rows, cols, ld, kPanelC, kPanelK, false);
    if (st != SF_OK) return st;
    const int resident = sms[dev] * kColsCtasPerSm;
    const unsigned grid = (unsigned)(num_panels < resident ? num_panels : resident);
    if (prune_mode == 0)
      prune24_cols_kernel<false><<<grid, 256, kColsSmemBytes, s>>>(tm, rows, cols, (uint16_t*)vals, (uint16_t*)meta,
                                                                   (uint8_t*)meta_hw, (uint16_t*)dense_out, (int)px, num_panels);
    else
      prune24_cols_kernel<true><<<grid, 256, kColsSmemBytes, s>>>(tm, rows, cols, (uint16_t*)vals, (uint16_t*)meta,
                                                                  (uint8_t*)meta_hw, (uint16_t*)dense_out, (int)px, num_panels);
  }
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int launch_prune24_cols_fp8(const void* W, int64_t rows, int64_t cols, int64_t ld, int prune_mode, float scale, void* vals,
                            void* meta, cudaStream_t s) {
  if (rows == 0 || cols == 0) return SF_OK;
  const int64_t px = (cols + kPanelC - 1) / kPanelC, py = (rows + kPanelK - 1) / kPanelK;
  if (px * py > (int64_t)1 << 30) return SF_ERR_SHAPE;
  const int num_panels = (int)(px * py);
  static bool attr_done[64] = {false};
  static int sms[64] = {0};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SF_ERR_UNSUPPORTED;
  if (!attr_done[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(prune24_cols_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColsSmemBytes));
    SF_CUDA_TRY(cudaFuncSetAttribute(prune24_cols_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kColsSmemBytes));
    SF_CUDA_TRY(cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev));
    attr_done[dev] = true;
  }
  alignas(64) CUtensorMap tm;
  int st = make_tmap_2d(&tm, W, rows, cols, ld, kPanelC, kPanelK, false);
  if (st != SF_OK) return st;
  const int resident = sms[dev] * kColsCtasPerSm;
  const unsigned grid = (unsigned)(num_panels < resident ? num_panels : resident);
  if (prune_mode == 0)
    prune24_cols_kernel<false, true><<<grid, 256, kColsSmemBytes, s>>>(tm, rows, cols, (uint16_t*)vals, (uint16_t*)meta, nullptr,
                                                                       nullptr, (int)px, num_panels, scale);
  else
    prune24_cols_kernel<true, true><<<grid, 256, kColsSmemBytes, s>>>(tm, rows, cols, (uint16_t*)vals, (uint16_t*)meta, nullptr,
                                                                      nullptr, (int)px, num_panels, scale);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int launch_transpose(const void* in, void* out, int64_t rows, int64_t cols, cudaStream_t s) {
  if (rows == 0 || cols == 0) return SF_OK;
  dim3 grid((unsigned)((cols + 63) / 64), (unsigned)((rows + 63) / 64));
  if (rows % 64 == 0 && cols % 64 == 0)
    transpose64_kernel<<<grid, 256, 0, s>>>((const uint16_t*)in, (uint16_t*)out, rows, cols);
  else
    transpose_kernel<<<grid, 256, 0, s>>>((const uint16_t*)in, (uint16_t*)out, rows, cols);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

}  // namespace sf
