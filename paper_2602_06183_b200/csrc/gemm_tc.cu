// Tensor-core products of the FFN step on sm_100a: tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA, warp-specialised roles.
//
//   mode DENSE     D[M,N] = A[M,K] B[N,K]^T                       (Eqs. 1-8; weight-gradient products)
//   mode SPARSE24  A is 2:4-compressed (values [M,K/2] + metadata) (Algorithm 1 line 4, Algorithm 2 line 2)
//   mode VENOM     A is V:N:M-compressed; B rows are gathered by the block's kept columns
//                  (Algorithm 1 line 7, Algorithm 2 line 5)
//
// CTA = 6 warps: warp 0 TMA producer, warp 1 MMA issuer (+ TMEM owner), warps 2-5 epilogue (each
// owns the 32 TMEM lanes of its quadrant). Tile 128 x 256, persistent over tiles (m fastest).
// Venom mode adds warps 6-17, which gather the kept rows of B into the 128B-swizzled MN-major
// layout the MMA reads: 8 warps issue TMA row gathers, 4 warps issue 16-byte cp.async copies.
// A stage holds A (16 KB dense, 8 KB compressed), B (32 KB) and, for sparse modes, one 2 KB metadata
// atom covering 128 rows x 128 logical K (copied smem -> TMEM by tcgen05.cp every second stage);
// 4 stages dense, 5 stages sparse.
// Dense mode double-buffers the 256-column accumulator so the epilogue of tile i overlaps the main
// loop of tile i+1; sparse modes keep one accumulator plus the metadata columns.
// Every mbarrier wait is bounded; on expiry the CTA raises a flag in the status word and leaves.
#include "sf_common.cuh"
#include "tc_ptx.cuh"
#include "gemm_tc.cuh"
#include "sparse_fmt.cuh"

namespace sf {

namespace {

using namespace ptx;

constexpr int BM = 128, BN = 256;
constexpr int kMaxStages = 5;
constexpr int kBStageBytes = 32768, kMetaStageBytes = 2048;
// dense: A 16 KB + B 32 KB, 4 stages; sparse modes: A 8 KB (stored half) + B 32 KB + metadata 2 KB, 5 stages
__host__ __device__ constexpr int a_stage_bytes(bool sparse) { return sparse ? 8192 : 16384; }
__host__ __device__ constexpr int stage_bytes(bool sparse) {
  return a_stage_bytes(sparse) + kBStageBytes + (sparse ? kMetaStageBytes : 0);
}
__host__ __device__ constexpr int num_stages(bool sparse) { return sparse ? 5 : 4; }
constexpr int kEpiStageRow = 80;                                                      // bytes: 32 bf16 + 16 pad
constexpr int kEpiStageBytes = 4 * 32 * kEpiStageRow;                                 // 4 warps
__host__ __device__ constexpr int smem_bytes(bool sparse) {
  return 1024 /*align slack*/ + num_stages(sparse) * stage_bytes(sparse) + kEpiStageBytes + 256 /*barriers*/;
}
constexpr int kThreads = 192;                 // dense / 2:4 modes: producer, MMA, 4 epilogue warps
constexpr int kThreadsVenom = 576;            // + 8 TMA-gather warps and 4 cp.async-gather warps
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kMetaTmemCol = 256;

struct SmemCtl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

// Tile raster: bands of kRasterM tile rows, m fastest inside a band. The tiles that run at the same
// time then form a near-square block (8 x ~9 for 74 CTA pairs), so a wave touches ~17 operand
// panels instead of ~65 and operands larger than the L2 are not re-read once per tile column.
constexpr int kRasterM = 8;
__device__ __forceinline__ void tile_coords(int tile, int num_m, int num_n, int& mt, int& nt) {
  const int per_band = kRasterM * num_n;
  const int band = tile / per_band, rem = tile - band * per_band;
  const int m_start = band * kRasterM;
  const int gm = min(kRasterM, num_m - m_start);
  nt = rem / gm;
  mt = m_start + (rem - nt * gm);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return float_to_bf16_bits(lo) | (float_to_bf16_bits(hi) << 16);
}


// ---- epilogue (shared by the one-CTA and the two-CTA kernels) ---------------------------------------
// One epilogue warp owns TMEM lanes [32q, 32q+32) of a 128 x 256 accumulator tile whose first row is
// m0 and first column n0; `taddr` is the TMEM address of (lane 32q, column 0) of that accumulator.
// kTileN: accumulator columns of the tile (a multiple of 32). Columns at or beyond args.N (a ragged last
// tile, whole 32-column chunks only since N % 32 == 0) are neither prefetched nor stored.
__host__ __device__ constexpr bool is_drelu_t(int epi) { return epi == EPI_DRELU_T || epi == EPI_DRELU24_T; }

template <int kEpi, int kTileN = BN>
__device__ __forceinline__ void epi_prefetch(const GemmArgs& args, int64_t m0, int64_t n0, int64_t n_limit, int q, int lane,
                                             uint4 (&ax)[is_drelu_t(kEpi) ? kTileN / 32 : 1][4]) {
  if (kEpi == EPI_DRELU24_T) {
    // ReLU(y1) in the 2:4 layout of the activation mask: four stored values and two position nibbles per
    // eight features; (x, y) = values, z = nibbles
#pragma unroll
    for (int ch = 0; ch < kTileN / 32; ++ch) {
      if (n0 + ch * 32 >= n_limit) break;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int64_t token = n0 + ch * 32 + i * 8 + (lane >> 2), f = m0 + q * 32 + (lane & 3) * 8;
        const uint2 r = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(args.aux) +
                                                             token * (args.M >> 1) + (f >> 1)));
        const uint32_t mb = __ldg(reinterpret_cast<const uint8_t*>(args.pack_meta) + token * (args.M >> 3) + (f >> 3));
        ax[is_drelu_t(kEpi) ? ch : 0][i] = make_uint4(r.x, r.y, mb, 0u);
      }
    }
  }
  if (kEpi == EPI_DRELU_T) {
#pragma unroll
    for (int ch = 0; ch < kTileN / 32; ++ch) {
      if (n0 + ch * 32 >= n_limit) break;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        ax[kEpi == EPI_DRELU_T ? ch : 0][i] = __ldg(reinterpret_cast<const uint4*>(
            reinterpret_cast<const uint16_t*>(args.aux) + (n0 + ch * 32 + i * 8 + (lane >> 2)) * args.ldaux + m0 +
            q * 32 + (lane & 3) * 8));
    }
  }
}

template <int kEpi, int kTileN = BN>
__device__ __forceinline__ void epi_tile(const GemmArgs& args, uint32_t taddr, int64_t m0, int64_t n0, int64_t n_limit,
                                         int q, int lane, uint8_t* my_stage,
                                         const uint4 (&ax)[is_drelu_t(kEpi) ? kTileN / 32 : 1][4]) {
  int64_t row = m0 + q * 32 + lane;                                        // this thread's D row
  if constexpr (kEpi == EPI_ROUTE) {
    // the row is a token, the first route_E columns its logits
    uint32_t v[32];
    tmem_ld_32x32b_x32(taddr, v);
    tmem_ld_wait_on(v);
    const int E = args.route_E;
    int best = 0;
    float bestv = __uint_as_float(v[0]);
#pragma unroll
    for (int e = 1; e < 16; ++e) {
      const float x = __uint_as_float(v[e]);
      if (e < E && x > bestv) { bestv = x; best = e; }                     // strict: ties stay with the lower expert
    }
    args.route_expert[row] = best;
    if (args.route_logits) {
#pragma unroll
      for (int e = 0; e < 16; ++e)
        if (e < E) args.route_logits[row * E + e] = __uint_as_float(v[e]);
    }
    return;
  }
  bool row_live = true;
  if (kEpi == EPI_STORE && args.row_map) {                                 // scattered output rows
    const int r = __ldg(args.row_map + row);
    row_live = r >= 0;
    row = r;
  }
  auto chunk = [&](int ch, const uint4 (&a4)[4], const uint32_t (&v)[32]) {
    const int64_t col0 = n0 + ch * 32;
    if (col0 >= n_limit) return;                                           // ragged last tile (warp-uniform)
    if (kEpi == EPI_STORE || kEpi == EPI_SQRELU || kEpi == EPI_DRELU) {
      uint16_t* crow = reinterpret_cast<uint16_t*>(args.C) + row * args.ldc + col0;
      if (kEpi == EPI_STORE) {
        if (!row_live) return;
        const float al = args.out_scale != 0.f ? args.out_scale : 1.f;      // x 1 is exact: bf16 products unchanged
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint4 o;
          o.x = pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * j + 0]), al), __fmul_rn(__uint_as_float(v[8 * j + 1]), al));
          o.y = pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * j + 2]), al), __fmul_rn(__uint_as_float(v[8 * j + 3]), al));
          o.z = pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * j + 4]), al), __fmul_rn(__uint_as_float(v[8 * j + 5]), al));
          o.w = pack_bf16x2(__fmul_rn(__uint_as_float(v[8 * j + 6]), al), __fmul_rn(__uint_as_float(v[8 * j + 7]), al));
          reinterpret_cast<uint4*>(crow)[j] = o;
        }
      } else if (kEpi == EPI_SQRELU) {
        uint16_t* hrow = reinterpret_cast<uint16_t*>(args.C2) + row * args.ldc2 + col0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t y[4], h[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t y0 = float_to_bf16_bits(__uint_as_float(v[8 * j + 2 * e]));
            const uint32_t y1 = float_to_bf16_bits(__uint_as_float(v[8 * j + 2 * e + 1]));
            const float f0 = fmaxf(bf16_bits_to_float(y0), 0.f), f1 = fmaxf(bf16_bits_to_float(y1), 0.f);
            y[e] = y0 | (y1 << 16);
            h[e] = pack_bf16x2(__fmul_rn(f0, f0), __fmul_rn(f1, f1));
          }
          reinterpret_cast<uint4*>(crow)[j] = make_uint4(y[0], y[1], y[2], y[3]);
          reinterpret_cast<uint4*>(hrow)[j] = make_uint4(h[0], h[1], h[2], h[3]);
        }
      } else {  // EPI_DRELU: C = bf16(2 * acc * relu(aux))
        const uint16_t* arow = reinterpret_cast<const uint16_t*>(args.aux) + row * args.ldaux + col0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 a = __ldg(reinterpret_cast<const uint4*>(arow) + j);
          const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
          uint32_t o[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float r0 = fmaxf(bf16_bits_to_float(aw[e] & 0xFFFFu), 0.f);
            const float r1 = fmaxf(bf16_bits_to_float(aw[e] >> 16), 0.f);
            const float d0 = __fmul_rn(__fmul_rn(2.f, __uint_as_float(v[8 * j + 2 * e])), r0);
            const float d1 = __fmul_rn(__fmul_rn(2.f, __uint_as_float(v[8 * j + 2 * e + 1])), r1);
            o[e] = pack_bf16x2(d0, d1);
          }
          reinterpret_cast<uint4*>(crow)[j] = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    } else {
      // Transposed output: D row = feature (lane), D column = token. C is [N, M] row-major.
      float r[32];
      // optional packed copy: the metadata words of this chunk's 32 tokens (features m0 + 32q .. + 31)
      const bool pack = kEpi == EPI_DRELU24_T || (kEpi == EPI_DRELU_T && args.pack_vals != nullptr);
      uint32_t mw[4] = {0, 0, 0, 0};
      if (pack && kEpi == EPI_DRELU_T) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          mw[i] = __ldg(reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint8_t*>(args.pack_meta) +
                                                         (col0 + i * 8 + (lane >> 2)) * (args.M >> 3) +
                                                         ((m0 + q * 32) >> 3)));
      }
      if (is_drelu_t(kEpi)) {
        // aux[token, feature] chunk -> staging -> one column per lane
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4*>(my_stage + (i * 8 + (lane >> 2)) * kEpiStageRow + (lane & 3) * 16) =
              kEpi == EPI_DRELU24_T ? expand24_x8(make_uint2(a4[i].x, a4[i].y), a4[i].z) : a4[i];
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 32; ++j)
          r[j] = bf16_bits_to_float(*reinterpret_cast<const uint16_t*>(my_stage + j * kEpiStageRow + lane * 2));
      }
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        float x = __uint_as_float(v[j]);
        uint32_t b;
        if (is_drelu_t(kEpi)) {
          // aux holds ReLU(y1) on the activation mask and +0 elsewhere: off-mask entries become +0
          b = (r[j] == 0.f) ? 0u : float_to_bf16_bits(__fmul_rn(__fmul_rn(2.f, x), r[j]));
        } else {
          b = float_to_bf16_bits(x);
        }
        *reinterpret_cast<uint16_t*>(my_stage + j * kEpiStageRow + lane * 2) = (uint16_t)b;
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = i * 8 + (lane >> 2), seg = lane & 3;
        const uint4 o = *reinterpret_cast<const uint4*>(my_stage + t * kEpiStageRow + seg * 16);
        if (kEpi == EPI_ACT24_T) {
          // o = y1 of eight neighbouring features of one token: SquaredReLU, then the two larger of every four
          const int64_t token = col0 + t, fl = m0 + q * 32 + seg * 8, Fe = args.M;
          const uint32_t r0w = bf2_relu(o.x), r1w = bf2_relu(o.y), r2w = bf2_relu(o.z), r3w = bf2_relu(o.w);
          uint32_t pa, pb;
          const uint32_t na = top2of4_packed(bf2_sq(r0w), bf2_sq(r1w), &pa), nb = top2of4_packed(bf2_sq(r2w), bf2_sq(r3w), &pb);
          const uint32_t ra = __byte_perm(r0w, r1w, 0x1010u + (na & 3u) * 0x22u + (na >> 2) * 0x2200u);
          const uint32_t rb = __byte_perm(r2w, r3w, 0x1010u + (nb & 3u) * 0x22u + (nb >> 2) * 0x2200u);
          const int64_t pv = (token * (Fe >> 1) + (fl >> 1)) >> 2;             // 8-byte units
          reinterpret_cast<uint2*>(args.vn_vals24)[pv] = make_uint2(pa, pb);
          reinterpret_cast<uint2*>(args.vn_relu24)[pv] = make_uint2(ra, rb);
          uint32_t mb = na | (nb << 4);
          reinterpret_cast<uint4*>(args.vn_dense)[(token * Fe + fl) >> 3] = expand24_x8(make_uint2(pa, pb), mb);
          if (args.vn_y1) reinterpret_cast<uint4*>(args.vn_y1)[(token * Fe + fl) >> 3] = o;
          // metadata: one byte per lane, four neighbouring lanes hold the warp's 32 features of this token
          mb |= __shfl_down_sync(0xFFFFFFFFu, mb, 1) << 8;
          const uint32_t mb32 = (mb & 0xFFFFu) | (__shfl_down_sync(0xFFFFFFFFu, mb, 2) << 16);
          const int64_t kw = (m0 + q * 32) >> 4;
          if (seg == 0) reinterpret_cast<uint32_t*>(args.vn_meta24)[(token * (Fe >> 4) + kw) >> 1] = mb32;
          if ((seg & 1) == 0)
            *reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(args.vn_meta24_hw) +
                                         meta_hw_offset(token, kw + (seg >> 1), Fe)) = (uint16_t)mb;
          continue;
        }
        if (kEpi != EPI_DRELU24_T || args.C != nullptr)
          *reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(args.C) + (col0 + t) * args.ldc + m0 + q * 32 + seg * 8) = o;
        if (pack) {
          // this lane's eight features are two groups of four: keep the two recorded positions of each
          const uint32_t mb = kEpi == EPI_DRELU24_T ? (a4[i].z & 0xFFu) : ((mw[i] >> (8 * seg)) & 0xFFu);
          const uint32_t p0 = __byte_perm(o.x, o.y, 0x1010u + (mb & 3u) * 0x22u + ((mb >> 2) & 3u) * 0x2200u);
          const uint32_t p1 = __byte_perm(o.z, o.w, 0x1010u + ((mb >> 4) & 3u) * 0x22u + (mb >> 6) * 0x2200u);
          *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(args.pack_vals) + (col0 + t) * (args.M >> 1) +
                                    ((m0 + q * 32 + seg * 8) >> 1)) = make_uint2(p0, p1);
        }
      }
    }
        };
  // Two register buffers: the TMEM load of the next 32 columns is in flight while this one is converted.
  uint32_t va[32], vb[32];
  tmem_ld_32x32b_x32(taddr, va);
  constexpr int kChunks = kTileN / 32;
  if (is_drelu_t(kEpi)) {
#pragma unroll
    for (int ch = 0; ch < kChunks; ch += 2) {
      tmem_ld_wait_on(va);
      if (ch + 1 < kChunks) tmem_ld_32x32b_x32(taddr + (ch + 1) * 32, vb);
      chunk(ch, ax[is_drelu_t(kEpi) ? ch : 0], va);
      if (ch + 1 < kChunks) {
        tmem_ld_wait_on(vb);
        if (ch + 2 < kChunks) tmem_ld_32x32b_x32(taddr + (ch + 2) * 32, va);
        chunk(ch + 1, ax[is_drelu_t(kEpi) ? (ch + 1 < kChunks ? ch + 1 : ch) : 0], vb);
      }
    }
  } else if (kChunks % 2 == 0) {
#pragma unroll 1
    for (int ch = 0; ch < kChunks; ch += 2) {
      tmem_ld_wait_on(va);
      tmem_ld_32x32b_x32(taddr + (ch + 1) * 32, vb);
      chunk(ch, ax[0], va);
      tmem_ld_wait_on(vb);
      if (ch + 2 < kChunks) tmem_ld_32x32b_x32(taddr + (ch + 2) * 32, va);
      chunk(ch + 1, ax[0], vb);
    }
  } else {
#pragma unroll
    for (int ch = 0; ch < kChunks; ch += 2) {
      tmem_ld_wait_on(va);
      if (ch + 1 < kChunks) tmem_ld_32x32b_x32(taddr + (ch + 1) * 32, vb);
      chunk(ch, ax[0], va);
      if (ch + 1 < kChunks) {
        tmem_ld_wait_on(vb);
        if (ch + 2 < kChunks) tmem_ld_32x32b_x32(taddr + (ch + 2) * 32, va);
        chunk(ch + 1, ax[0], vb);
      }
    }
  }
}


// ---- fused SquaredReLU + V:N:M selection (groups of eight) ---------------------------------------------
// Epilogue of the y1 product: the accumulator tile is y1^T (TMEM lane = feature, column = token), so a
// lane owns one feature column of every V x 8 block and eight neighbouring lanes own one block.
// Per V-block of the tile, each epilogue warp (32 features = four groups):
//   pass 1  reads its lanes' V accumulator columns, rounds them to bf16 (this is y1), parks them in
//           shared memory as [token][feature], and accumulates the column score of Section 2.3 in
//           float32, token by token in ascending order (the order is part of the format);
//   rank    the eight lanes of a group exchange scores; the four best columns stay (ties to the lower
//           column), their indices go to colidx and into per-group byte-permute selector tables;
//   pass 2  one thread per (token, group) takes the group's eight values back from shared memory, applies
//           SquaredReLU, keeps the two largest of the four kept columns and writes the packed activation,
//           the packed ReLU values, both metadata forms and the 2:4 view.
// The accumulator is released to the MMA warp as soon as the last block's pass 1 has read it.
// Shared memory of one epilogue warp: y1 of one block as [token pair][feature] words (low half = even
// token), then colidx, the selector table and the nibble table of the block.
__host__ __device__ constexpr int vnm_stage_bytes(int V) { return V * 64; }
__host__ __device__ constexpr int vnm_warp_bytes(int V) { return vnm_stage_bytes(V) + 16 + 4 * 7 * 16 + 48; }
constexpr int kVnmEpiWarps = 8;                                  // two sets of four: one set per accumulator buffer
__host__ __device__ constexpr int vnm_epi_bytes(int V) { return kVnmEpiWarps * vnm_warp_bytes(V); }

template <int kTileN, int kV>
__device__ __forceinline__ void epi_vnm8_tile(const GemmArgs& args, uint32_t taddr, int64_t m0, int64_t n0,
                                              int64_t n_limit, int q, int lane, uint8_t* wsm, uint64_t* tmem_empty_bar) {
  uint32_t* stage = reinterpret_cast<uint32_t*>(wsm);                     // [kV / 2][32 features]
  uint8_t* cidx = wsm + vnm_stage_bytes(kV);                              // [4 groups][4]
  uint4* sel_tab = reinterpret_cast<uint4*>(wsm + vnm_stage_bytes(kV) + 16);   // [4 groups][7]
  uint8_t* nib_tab = wsm + vnm_stage_bytes(kV) + 16 + 4 * 7 * 16;         // [4 groups][7]
  const int64_t F = args.M, G = F >> 3;
  const int64_t f0 = m0 + q * 32, g0 = f0 >> 3;                           // this warp's first feature / group
  const int jm = lane & 7, gl = lane & 3;
  constexpr int kBlocks = kTileN / kV;
  int nblk = kBlocks;
  while (nblk > 0 && n0 + (int64_t)(nblk - 1) * kV >= n_limit) --nblk;     // ragged last tile: whole blocks only
  if (nblk == 0) {
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive_leader(tmem_empty_bar);
    return;
  }
  // strides per token of the outputs this thread writes (in the units of its pointers)
  const int sv = (int)G, s24 = (int)(F >> 3), sm = (int)(G >> 2), sm24 = (int)(F >> 5);
  const bool lead4 = gl == 0, lead2 = (gl & 1) == 0;
#pragma unroll 1
  for (int b = 0; b < kBlocks; ++b) {
    if (b >= nblk) break;
    __syncwarp();                                                          // the previous block's pass 2 has read the stage
    const int64_t t0 = n0 + (int64_t)b * kV;
    // ---- pass 1: two tokens per step on packed bf16 pairs
    float score = 0.f;
    uint32_t v[32];
#pragma unroll 1
    for (int c = 0; c < kV / 32; ++c) {
      tmem_ld_32x32b_x32(taddr + (uint32_t)(b * kV + c * 32), v);
      tmem_ld_wait_on(v);
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t yp = pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
        stage[(c * 16 + j) * 32 + lane] = yp;
        const uint32_t hp = bf2_sq(bf2_relu(yp));
        score = __fadd_rn(score, __uint_as_float(hp << 16));
        score = __fadd_rn(score, __uint_as_float(hp & 0xFFFF0000u));
      }
    }
    if (b == nblk - 1) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(tmem_empty_bar);
    }
    // ---- rank the eight columns of each group
    const uint32_t sb = __float_as_uint(score);                            // scores are >= 0: the pattern orders them
    int rank = 0;
#pragma unroll
    for (int i = 1; i < 8; ++i) {
      const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, sb, i);
      const int oj = jm ^ i;
      rank += (o > sb) || (o == sb && oj < jm);
    }
    const bool keep = rank < 4;
    const uint32_t ball = __ballot_sync(0xFFFFFFFFu, keep);
    const uint32_t gbyte = (ball >> (lane & 24)) & 0xFFu;
    if (keep) cidx[(lane >> 3) * 4 + __popc(gbyte & ((1u << jm) - 1u))] = (uint8_t)jm;
    __syncwarp();
    if (lane < 4)
      *reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(args.vn_colidx) + ((t0 / kV) * G + g0 + lane) * 4) =
          *reinterpret_cast<const uint32_t*>(cidx + lane * 4);
    if (lane < 24) {
      const int ge = lane / 6, pe = lane - ge * 6;
      const int pi = pe < 3 ? 0 : (pe < 5 ? 1 : 2), pj = pe < 3 ? pe + 1 : (pe < 5 ? pe - 1 : 3);
      uint4 selv;
      uint32_t nib24;
      vnm8_pair_selectors(cidx[ge * 4 + pi], cidx[ge * 4 + pj], selv, nib24);
      const int slot = ge * 7 + (int)nib_slot((uint32_t)pi | ((uint32_t)pj << 2));
      sel_tab[slot] = selv;
      nib_tab[slot] = (uint8_t)nib24;
    }
    __syncwarp();
    // ---- pass 2: this thread serves group gl of the token pairs (lane >> 2) + 8 * it
    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + gl * 4);
    uint32_t selp[2], mhi[2];
#pragma unroll
    for (int pr = 0; pr < 2; ++pr) {
      const uint32_t ca = (c4 >> (16 * pr)) & 0xFFu, cb = (c4 >> (16 * pr + 8)) & 0xFFu;
      const uint32_t sa = 2u * (ca & 3u), sbb = 2u * (cb & 3u);
      selp[pr] = sa | ((sa + 1u) << 4) | (sbb << 8) | ((sbb + 1u) << 12);
      mhi[pr] = ((ca & 4u) ? 0x0000FFFFu : 0u) | ((cb & 4u) ? 0xFFFF0000u : 0u);
    }
    const uint4* my_sel = sel_tab + gl * 7;
    const uint8_t* my_nib = nib_tab + gl * 7;
    // output pointers of this thread's first token; every pointer advances by a constant per token
    const int64_t tf = t0 + 2 * (lane >> 2);
    uint32_t* p_vals = reinterpret_cast<uint32_t*>(args.vn_vals) + tf * G + g0 + gl;
    uint32_t* p_relu = reinterpret_cast<uint32_t*>(args.vn_relu) + tf * G + g0 + gl;
    uint2* p_v24 = reinterpret_cast<uint2*>(args.vn_vals24) + tf * (F >> 3) + g0 + gl;
    uint2* p_r24 = reinterpret_cast<uint2*>(args.vn_relu24) + tf * (F >> 3) + g0 + gl;
    uint4* p_y1 = args.vn_y1 ? reinterpret_cast<uint4*>(args.vn_y1) + tf * (F >> 3) + g0 + gl : nullptr;
    uint4* p_dense = args.vn_dense ? reinterpret_cast<uint4*>(args.vn_dense) + tf * (F >> 3) + g0 + gl : nullptr;
    uint16_t* p_meta = reinterpret_cast<uint16_t*>(args.vn_meta) + tf * (G >> 2) + (g0 >> 2);
    uint32_t* p_m24 = reinterpret_cast<uint32_t*>(args.vn_meta24) + tf * (F >> 5) + (f0 >> 5);
    // tensor-core-ordered copy: the block lies inside one 128-row band, so the atom is fixed
    const int64_t kw24 = (f0 >> 4) + (gl >> 1);
    uint8_t* hw_atom = reinterpret_cast<uint8_t*>(args.vn_meta24_hw) + meta_hw_offset(t0 & ~int64_t(127), kw24, F);
    const uint32_t* sp = stage + (lane >> 2) * 32 + gl * 8;

    auto emit = [&](const uint32_t (&yw)[4], int dt, uint32_t trow) {
      uint32_t rw[4], hw[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) { rw[j] = bf2_relu(yw[j]); hw[j] = bf2_sq(rw[j]); }
      const uint32_t a0 = __byte_perm(hw[0], hw[1], selp[0]), b0 = __byte_perm(hw[2], hw[3], selp[0]);
      const uint32_t a1 = __byte_perm(hw[0], hw[1], selp[1]), b1 = __byte_perm(hw[2], hw[3], selp[1]);
      const uint32_t hk0 = (a0 & ~mhi[0]) | (b0 & mhi[0]), hk1 = (a1 & ~mhi[1]) | (b1 & mhi[1]);
      uint32_t packed;
      const uint32_t nib = top2of4_packed(hk0, hk1, &packed);
      const uint32_t slot = nib_slot(nib);
      const uint4 sel = my_sel[slot];
      const uint32_t x = __byte_perm(rw[0], rw[1], sel.z), y = __byte_perm(rw[2], rw[3], sel.z);
      const uint32_t rpair = __byte_perm(x, y, sel.z >> 16);
      p_vals[dt * sv] = packed;
      p_relu[dt * sv] = rpair;
      p_v24[dt * s24] = make_uint2(__byte_perm(packed, 0u, sel.w), __byte_perm(packed, 0u, sel.w >> 16));
      p_r24[dt * s24] = make_uint2(__byte_perm(rpair, 0u, sel.w), __byte_perm(rpair, 0u, sel.w >> 16));
      if (p_y1) p_y1[dt * s24] = make_uint4(yw[0], yw[1], yw[2], yw[3]);
      if (p_dense)
        p_dense[dt * s24] = make_uint4(__byte_perm(packed, 0u, sel.x), __byte_perm(packed, 0u, sel.x >> 16),
                                       __byte_perm(packed, 0u, sel.y), __byte_perm(packed, 0u, sel.y >> 16));
      // canonical V:N:M metadata: the warp's four groups of a token form one word
      uint32_t word = nib;
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 4;
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 8;
      if (lead4) p_meta[dt * sm] = (uint16_t)word;
      // metadata of the 2:4 view: one byte per group, one 16-bit word per pair of groups
      uint32_t mb = my_nib[slot];
      mb |= __shfl_down_sync(0xFFFFFFFFu, mb, 1) << 8;
      const uint32_t mb32 = (mb & 0xFFFFu) | (__shfl_down_sync(0xFFFFFFFFu, mb, 2) << 16);
      if (lead4) p_m24[dt * sm24] = mb32;
      if (lead2) {
        const uint32_t mi = trow & 127u;
        *reinterpret_cast<uint16_t*>(hw_atom + (mi >> 4) * 256u + (mi & 7u) * 16u + ((mi >> 3) & 1u) * 2u) = (uint16_t)mb;
      }
    };
    // A quarter-warp reads two token pairs x four groups; pairs alternate which 16-byte half they fetch
    // first, so each of the two loads touches every bank exactly once.
    const int swap = (lane >> 2) & 1;
#pragma unroll 1
    for (int it = 0; it < kV / 16; ++it) {
      const uint4 q0 = *reinterpret_cast<const uint4*>(sp + 4 * swap), q1 = *reinterpret_cast<const uint4*>(sp + 4 - 4 * swap);
      const uint4 qa = swap ? q1 : q0, qb = swap ? q0 : q1;
      // de-interleave the token pair: low halves = even token, high halves = odd token
      const uint32_t r0[4] = {__byte_perm(qa.x, qa.y, 0x5410), __byte_perm(qa.z, qa.w, 0x5410),
                              __byte_perm(qb.x, qb.y, 0x5410), __byte_perm(qb.z, qb.w, 0x5410)};
      const uint32_t r1[4] = {__byte_perm(qa.x, qa.y, 0x7632), __byte_perm(qa.z, qa.w, 0x7632),
                              __byte_perm(qb.x, qb.y, 0x7632), __byte_perm(qb.z, qb.w, 0x7632)};
      const uint32_t trow = (uint32_t)(tf & 127) + 16u * (uint32_t)it;
      emit(r0, 0, trow);
      emit(r1, 1, trow + 1u);
      sp += 8 * 32;
      p_vals += 16 * sv; p_relu += 16 * sv; p_v24 += 16 * s24; p_r24 += 16 * s24;
      if (p_y1) p_y1 += 16 * s24;
      if (p_dense) p_dense += 16 * s24;
      p_meta += 16 * sm; p_m24 += 16 * sm24;
    }
  }
}

template <int kMode, bool kAMN, bool kBMN, int kEpi>
__global__ void __launch_bounds__(kMode == MODE_VENOM ? kThreadsVenom : kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
               const GemmArgs args) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  constexpr bool kSparse = kMode != MODE_DENSE;
  constexpr int kStages = num_stages(kSparse);
  constexpr int kAStageBytes = a_stage_bytes(kSparse);
  constexpr int kStageBytes = stage_bytes(kSparse);
  uint8_t* epi_stage = smem + kStages * kStageBytes;
  SmemCtl* ctl = reinterpret_cast<SmemCtl*>(epi_stage + kEpiStageBytes);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kAccBufs = kSparse ? 1 : 2;
  constexpr int kMmaPerStage = kSparse ? 2 : 4;      // dense: K=16 x4 = 64; sparse: logical K=32 x2 = 64

  const int num_m_tiles = args.num_m_tiles, num_n_tiles_ = args.num_n_tiles;
  const int num_tiles = num_m_tiles * num_n_tiles_;
  const int nkb = args.num_k_blocks;                 // 64-wide (logical) k blocks per sweep
  const int sweeps = (kMode == MODE_VENOM && args.V == 64) ? 2 : 1;
  const int iters = nkb * sweeps;

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmapA);
    prefetch_tmap(&tmapB);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctl->full[s], kMode == MODE_VENOM ? 1 + 128 : 1);   // Venom: + one arrival per cp.async gather thread
      mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->tmem_full[b], 1);
      mbar_init(&ctl->tmem_empty[b], 4);
    }
    ctl->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&ctl->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // =========================== TMA producer ===========================
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int mt, nt;
      tile_coords(tile, num_m_tiles, num_n_tiles_, mt, nt);
      const int m0 = mt * BM, n0 = nt * BN;
      for (int it = 0; it < iters; ++it) {
        const int sweep = it / nkb, kb = it - sweep * nkb;
        if (!mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
        uint8_t* sA = smem + stage * kStageBytes;
        uint8_t* sB = sA + kAStageBytes;
        uint8_t* sM = sB + kBStageBytes;
        uint64_t* bar = &ctl->full[stage];
        const bool load_meta = kSparse && ((kb & 1) == 0);
        if (lane == 0) {
          const uint32_t b_tx = (kMode != MODE_VENOM) ? (uint32_t)kBStageBytes
                                                      : (uint32_t)args.gather_tma_groups * 2048u;  // TMA-gathered part
          uint32_t bytes = b_tx + (kSparse ? 8192u : 16384u) + (load_meta ? (uint32_t)kMetaStageBytes : 0u);
          mbar_arrive_expect_tx(bar, bytes);
          // ---- A
          if (kMode == MODE_DENSE) {
            if (!kAMN) {
              tma_load_2d(sA, &tmapA, bar, kb * 64, m0);                       // box {64 k, 128 m}
            } else {
              tma_load_2d(sA, &tmapA, bar, m0, kb * 64);                       // box {64 m, 64 k}
              tma_load_2d(sA + 8192, &tmapA, bar, m0 + 64, kb * 64);
            }
          } else if (kMode == MODE_SPARSE24 || sweeps == 1) {
            tma_load_2d(sA, &tmapA, bar, kb * 32, m0);                         // stored: box {32, 128}
          } else {
            // V = 64: this sweep owns one 64-row half of the tile; the other half reads the zero
            // fill of an out-of-range row coordinate. (box {32, 64})
            const int oob = (int)args.M + 64;
            tma_load_2d(sA, &tmapA, bar, kb * 32, sweep == 0 ? m0 : oob);
            tma_load_2d(sA + 4096, &tmapA, bar, kb * 32, sweep == 1 ? m0 + 64 : oob);
          }
          // ---- metadata atom (2 KB, contiguous in the hardware-ordered tensor)
          if (load_meta) {
            const uint8_t* src = args.meta_hw + ((size_t)mt * (size_t)(nkb >> 1) + (size_t)(kb >> 1)) * 2048;
            bulk_load(sM, src, kMetaStageBytes, bar);
          }
          // ---- B (non-gathered)
          if (kMode != MODE_VENOM) {
            if (!kBMN) {
              tma_load_2d(sB, &tmapB, bar, kb * 64, n0);                       // box {64 k, 256 n}
            } else {
#pragma unroll
              for (int c = 0; c < 4; ++c) tma_load_2d(sB + c * 8192, &tmapB, bar, n0 + c * 64, kb * 64);
            }
          }
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(BM, BN, kAMN, kBMN || kMode == MODE_VENOM, kSparse);
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(&ctl->tmem_empty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        for (int it = 0; it < iters; ++it) {
          const int kb = it % nkb;
          if (!mbar_wait(&ctl->full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sA = smem_u32(smem + stage * kStageBytes);
          const uint32_t sB = sA + kAStageBytes;
          const uint32_t sM = sB + kBStageBytes;
          if (kSparse && (kb & 1) == 0) {
            // 128 rows x 16 B, no swizzle: 8-row core matrices 128 B apart
            tmem_cp_128x128b(tmem_base + kMetaTmemCol + 4u * ((uint32_t)(kb >> 1) & 1u),
                             smem_desc(sM, 128, 128, kSwizzleNone));
          }
#pragma unroll
          for (int k = 0; k < kMmaPerStage; ++k) {
            uint64_t adesc, bdesc;
            if (kMode == MODE_DENSE) {
              adesc = kAMN ? smem_desc(sA + k * 2048, 8192, 1024, kSwizzle128B)
                           : smem_desc(sA + k * 32, 16, 1024, kSwizzle128B);
            } else {
              adesc = smem_desc(sA + k * 32, 16, 512, 4 /* 64 B swizzle */);
            }
            if (kMode == MODE_VENOM || kBMN) {
              // MN-major: 16 (dense) or 32 (sparse) k rows of 128 B per instruction
              bdesc = smem_desc(sB + k * (kSparse ? 4096 : 2048), 8192, 1024, kSwizzle128B);
            } else {
              bdesc = smem_desc(sB + k * (kSparse ? 64 : 32), 16, 1024, kSwizzle128B);
            }
            const uint32_t accum = (it > 0 || k > 0) ? 1u : 0u;
            if (kSparse) {
              const uint32_t col = (uint32_t)((kb & 1) * 2 + k);              // metadata column of this k step
              const uint32_t mbuf = kMetaTmemCol + 4u * ((uint32_t)(kb >> 1) & 1u);   // metadata double buffer
              mma_sp_f16(tmem_d, adesc, bdesc, tmem_base + mbuf + (col & ~1u), idesc | (col & 1u), accum);
            } else {
              mma_f16(tmem_d, adesc, bdesc, idesc, accum);
            }
          }
          mma_commit(&ctl->empty[stage]);                                      // frees the smem stage
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        mma_commit(&ctl->tmem_full[acc]);                                      // accumulator ready
        if (++acc == (uint32_t)kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else if (kMode == MODE_VENOM && warp >= 6) {
    // =========================== B gather (warps 6..17, Venom only) ===========================
    // Stage rows are the kept feature rows of Bt in condensed-k order: row r of the stage is
    // feature g*Mv + colidx[blk][g][r & 3] with g = kb*16 + r/4. Two engines work side by side:
    //   warps 6..13  TMA row gather (4 rows x 128 B per instruction) for the first `ntma` groups,
    //   warps 14..17 16-byte cp.async (one warp-wide copy = 512 B of one row) for the others.
    // Neither path alone keeps up with the tensor core; their in-flight limits are independent.
    const int gw = warp - 6;
    const int ntma = args.gather_tma_groups;
    const uint16_t* Bt = reinterpret_cast<const uint16_t*>(args.aux);
    uint32_t stage = 0, phase = 0;
    int pending = -1;                      // cp.async warps: stage whose copies are issued but not yet signalled
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int mt, nt;
      tile_coords(tile, num_m_tiles, num_n_tiles_, mt, nt);
      const int64_t n0 = (int64_t)nt * BN;
      for (int it = 0; it < iters; ++it) {
        const int sweep = it / nkb, kb = it - sweep * nkb;
        if (!mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
        const uint32_t sB = smem_u32(smem + stage * kStageBytes + kAStageBytes);
        const int blk = (args.V == 64) ? (2 * mt + sweep) : mt;
        const uint8_t* cbase = args.colidx + ((int64_t)blk * args.G + (int64_t)kb * 16) * 4;
        if (gw < 8) {
          const int grp = gw + 8 * (lane >> 2), c = lane & 3;             // lanes 0..7: two groups x 4 chunks
          if (lane < 8 && grp < ntma) {
            const uint32_t cg = *reinterpret_cast<const uint32_t*>(cbase + grp * 4);
            const int base = (int)(((int64_t)kb * 16 + grp) * args.Mv);
            tma_gather4_2d(sB + c * 8192 + grp * 4 * 128, &tmapB, &ctl->full[stage], (int)n0 + c * 64,
                           base + (int)(cg & 0xFF), base + (int)((cg >> 8) & 0xFF), base + (int)((cg >> 16) & 0xFF),
                           base + (int)(cg >> 24));
          }
        } else {
          const int cw = gw - 8;                                          // 0..3
          for (int grp = ntma + cw; grp < 16; grp += 4) {
            const uint32_t cg = *reinterpret_cast<const uint32_t*>(cbase + grp * 4);
            const int64_t fbase = ((int64_t)kb * 16 + grp) * args.Mv;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int row = grp * 4 + i;
              const uint16_t* src = Bt + (fbase + ((cg >> (8 * i)) & 0xFFu)) * args.ldaux + n0 + lane * 8;
              const uint32_t dst = sB + (lane >> 3) * 8192 + row * 128 + (((lane & 7) ^ (row & 7)) << 4);
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            }
          }
          asm volatile("cp.async.commit_group;" ::: "memory");
          // These copies are generic-proxy writes and the MMA reads the stage through the async proxy:
          // a stage is signalled only after its copies have landed and a proxy fence has ordered them.
          // The warps stay one stage ahead: signal the previous stage while this one is in flight.
          if (pending >= 0) {
            asm volatile("cp.async.wait_group 1;" ::: "memory");
            fence_proxy_async_smem();
            mbar_arrive(&ctl->full[pending]);
          }
          pending = (int)stage;
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    if (gw >= 8) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      if (pending >= 0) {
        fence_proxy_async_smem();
        mbar_arrive(&ctl->full[pending]);
      }
    }
  } else {
    // =========================== epilogue (warps 2..5) ===========================
    const int q = warp & 3;                                                    // TMEM lane quadrant
    uint8_t* my_stage = epi_stage + q * 32 * kEpiStageRow;
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int mt, nt;
      tile_coords(tile, num_m_tiles, num_n_tiles_, mt, nt);
      const int64_t m0 = (int64_t)mt * BM, n0 = (int64_t)nt * BN;
      // The dy1 epilogue multiplies by a [token, feature] tile of the saved activations; its loads do
      // not depend on the accumulator, so they are issued before the wait and land during the main loop.
      uint4 ax[is_drelu_t(kEpi) ? BN / 32 : 1][4];
      epi_prefetch<kEpi>(args, m0, n0, args.N, q, lane, ax);
      if (!mbar_wait(&ctl->tmem_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
      epi_tile<kEpi>(args, taddr, m0, n0, args.N, q, lane, my_stage, ax);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->tmem_empty[acc]);
      if (++acc == (uint32_t)kAccBufs) { acc = 0; acc_phase ^= 1; }
    }
  }

  // =========================== teardown ===========================
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctl->abort_flag) atomicExch(args.status, 1);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- two-CTA kernel (cta_group::2) -----------------------------------------------------------------
// A cluster of two CTAs computes one 256 x 256 tile: CTA r holds rows [128r, 128r+128) of A and of
// the accumulator, and columns [128r, 128r+128) of B; the leader (rank 0) issues MMAs that read both
// CTAs' shared memory. Each CTA therefore fetches half as much B per unit of tensor work as the
// one-CTA kernel. No TMA multicast is used: each CTA loads its own halves, with completion bytes
// routed to the leader's barrier.
// Stage = 64 K (dense, 4 MMAs of K=16) or 128 logical K (2:4, 4 MMAs of K=32 and one metadata atom):
// four MMAs per barrier round trip keep the single issuing thread ahead of the tensor pipe.
constexpr int kThreads2 = 192;
constexpr int kThreads2Expand = 448;                     // + eight warps that expand a packed operand into its stage
constexpr int kThreads2Vnm = 320;                        // + a second set of four epilogue warps (one set per accumulator)
__host__ __device__ constexpr int threads2(int epi, int expand) {
  return expand ? kThreads2Expand : (epi == EPI_VNM8 ? kThreads2Vnm : kThreads2);
}
constexpr int kPkStageBytes = 8192 + 1024;               // packed values [64 tokens][64] + metadata bytes [64][16]
// 8-bit operands (fp8 = true) keep the byte geometry of a stage (128-byte rows now hold 128 elements, so a
// 2:4 stage spans 256 logical K) and double its metadata: two 2 KB atoms.
__host__ __device__ constexpr int meta_stage_bytes2(bool fp8) { return fp8 ? 4096 : 2048; }
__host__ __device__ constexpr int stage_bytes2(bool sparse, int bn = BN, bool fp8 = false) {
  return sparse ? (16384 + 2 * (bn / 2) * 128 + meta_stage_bytes2(fp8)) : (16384 + 16384);
}
__host__ __device__ constexpr int num_stages2(bool sparse, int bn = BN, bool expand = false) {
  return sparse ? 4 : (expand ? 5 : 6);
}
// the fused activation epilogue holds whole V-blocks per tile: 192 columns = three blocks of 64, 128 = one of 128
__host__ __device__ constexpr int vnm_block(int bn) { return bn == 192 ? 64 : 128; }
__host__ __device__ constexpr int epi_bytes2(int epi, int bn = BN) {
  return epi == EPI_VNM8 ? vnm_epi_bytes(vnm_block(bn)) : kEpiStageBytes;
}
__host__ __device__ constexpr int smem_bytes2(bool sparse, int bn = BN, int epi = EPI_STORE, bool expand = false,
                                              bool fp8 = false) {
  return 1024 + num_stages2(sparse, bn, expand) * (stage_bytes2(sparse, bn, fp8) + (expand ? kPkStageBytes : 0)) +
         epi_bytes2(epi, bn) + 1024;
}

struct SmemCtl2 {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t pk_full[8];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint2 expand_lut[16];      // byte-permute selectors of a 2:4 nibble (see the operand expander)
  uint32_t tmem_base;
  int abort_flag;
};

// The tile a CTA pair works on: from the regular raster, or from a device-built table (grouped products).
template <int kBN>
__device__ __forceinline__ GemmTile get_tile(const GemmArgs& args, int tile, int num_m, int num_n, int nkb_full) {
  if (args.tile_table) {
    const int4* p = reinterpret_cast<const int4*>(args.tile_table + tile);
    const int4 a = __ldg(p), b = __ldg(p + 1);
    return GemmTile{a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
  }
  int mt, nt;
  tile_coords(tile, num_m, num_n, mt, nt);
  return GemmTile{mt * 256, 0, nt * kBN, 0, nkb_full, mt * 256, nt * kBN, (int)args.N};
}

__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi) {
  return (static_cast<uint64_t>(hi) << 32) | lo;
}

// kExpand (dense mode with both operands MN-major only): 1 = operand A, 2 = operand B is not loaded as a
// dense tile; its 2:4-packed form (tmapPk: values, tmapMeta: metadata bytes) is staged by TMA and four
// extra warps expand it, zero-filled, into the swizzled layout the MMA reads.
// kFp8: E4M3 operands (both K-major). The kernel is unchanged in bytes: K, k-block counts and operand
// coordinates are given in 2-byte units (two codes each); only the instruction kind, the descriptor's formats
// and the amount of metadata per stage differ.
template <int kMode, bool kAMN, bool kBMN, int kEpi, int kBN = BN, int kExpand = 0, bool kFp8 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(threads2(kEpi, kExpand), 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                const __grid_constant__ CUtensorMap tmapMeta, const __grid_constant__ CUtensorMap tmapPk,
                const GemmArgs args) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  constexpr bool kSparse = kMode == MODE_SPARSE24;
  constexpr int kStages = num_stages2(kSparse, kBN, kExpand != 0);
  constexpr int kBK = kSparse ? 128 : 64;                // logical K per stage
  static_assert(kExpand == 0 || (kMode == MODE_DENSE && kAMN && kBMN), "packed operands: weight-gradient products only");
  static_assert(!kFp8 || (!kAMN && !kBMN && kExpand == 0 && kMode != MODE_VENOM), "8-bit operands are K-major");
  constexpr int kMetaBytes = meta_stage_bytes2(kFp8);
  constexpr uint32_t kMetaCols = kFp8 ? 8u : 4u;          // TMEM columns of one stage's metadata
  constexpr int kAStageBytes = 16384;
  constexpr int kBSlabBytes = (kBN / 2) * 128;            // this CTA's half of B for one 64-wide K slab
  constexpr int kBHalfBytes = kSparse ? 2 * kBSlabBytes : kBSlabBytes;
  constexpr int kStageBytes = stage_bytes2(kSparse, kBN, kFp8);
  // 2:4 mode: TMEM holds the metadata next to the accumulators, so 256-column tiles leave room for one
  // accumulator only; 224-column tiles fit two (448 columns + 8 of metadata) and the epilogue of a tile
  // then overlaps the main loop of the next.
  constexpr int kAccBufs = (kSparse && kBN > 248) ? 1 : 2;
  constexpr uint32_t kMetaCol = kSparse ? (uint32_t)(kAccBufs * kBN) : 0u;
  static_assert(kBN % 32 == 0 && kBN <= 256, "tile width");
  static_assert(!(kMode == MODE_DENSE) || kBN == BN, "dense mode uses 256-column tiles");
  static_assert(!kBMN || kBN == BN, "MN-major B is loaded in 64-column chunks");
  uint8_t* pk_stage = smem + kStages * kStageBytes;       // kExpand: ring of packed tiles, one per stage
  uint8_t* epi_stage = pk_stage + (kExpand ? kStages * kPkStageBytes : 0);
  SmemCtl2* ctl = reinterpret_cast<SmemCtl2*>(epi_stage + epi_bytes2(kEpi, kBN));
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int num_m_tiles = args.num_m_tiles, num_n_tiles_ = args.num_n_tiles;   // 256-row tiles
  const int num_tiles = args.tile_table ? __ldg(args.num_tiles_dev) : num_m_tiles * num_n_tiles_;
  const int nkb_full = (int)(args.K / kBK);

  if (threadIdx.x == 0) {
    prefetch_tmap(&tmapA);
    prefetch_tmap(&tmapB);
    if (kSparse || kExpand) prefetch_tmap(&tmapMeta);
    if (kExpand) prefetch_tmap(&tmapPk);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctl->full[s], kExpand ? 1 + 16 : 1);    // + the eight expander warps of either CTA
      mbar_init(&ctl->empty[s], 1);
      mbar_init(&ctl->pk_full[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&ctl->tmem_full[b], 1);
      mbar_init(&ctl->tmem_empty[b], 8);                 // 4 epilogue warps in each CTA of the pair
    }
    ctl->abort_flag = 0;
    fence_mbar_init();
  }
  if (kExpand && threadIdx.x >= 64 && threadIdx.x < 80) {
    // nibble n = p0 | p1 << 2: output byte pair of column c takes stored value 0 (bytes 1,0) if c == p0,
    // value 1 (bytes 3,2) if c == p1, else the zero operand (byte 4)
    const uint32_t n = threadIdx.x - 64;
    const uint32_t sel = 0x44444444u ^ (0x54u << (8u * (n & 3u))) ^ (0x76u << (8u * (n >> 2)));
    ctl->expand_lut[n] = make_uint2(sel & 0xFFFFu, sel >> 16);
  }
  if (warp == 1) {
    tmem_alloc_2cta(&ctl->tmem_base, kTmemCols);
    tmem_relinquish_2cta();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                    // both CTAs' barriers and TMEM are ready
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // =========================== TMA producer (both CTAs) ===========================
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
      const GemmTile tc = get_tile<kBN>(args, tile, num_m_tiles, num_n_tiles_, nkb_full);
      const int m0 = tc.a_row + (int)rank * 128;         // this CTA's rows of A / D
      const int nb0 = tc.b_row + (int)rank * (kBN / 2);  // this CTA's columns of B
      const int nkb = tc.nkb, ak0 = tc.a_k0, bk0 = tc.b_k0;
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(&ctl->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
        if (lane == 0) {
          uint8_t* sA = smem + stage * kStageBytes;
          uint8_t* sB = sA + kAStageBytes;
          uint8_t* sM = sB + kBHalfBytes;
          uint64_t* bar = &ctl->full[stage];
          if (rank == 0) {
            // the leader's barrier collects the bytes of both CTAs (an expanded operand arrives by
            // shared-memory stores, not by TMA)
            mbar_arrive_expect_tx(bar, 2u * ((kExpand == 1 ? 0u : (uint32_t)kAStageBytes) +
                                             (kExpand == 2 ? 0u : (uint32_t)kBHalfBytes) +
                                             (kSparse ? (uint32_t)kMetaBytes : 0u)));
          }
          if (kMode == MODE_DENSE) {
            if (kExpand == 1) {
              // packed A: this CTA's 128 features of 64 tokens, into the staging ring (own barrier)
            } else if (!kAMN) {
              tma_load_2d_2cta(sA, &tmapA, bar, ak0 + kb * 64, m0);
            } else {
              tma_load_2d_2cta(sA, &tmapA, bar, m0, ak0 + kb * 64);
              tma_load_2d_2cta(sA + 8192, &tmapA, bar, m0 + 64, ak0 + kb * 64);
            }
            if (kExpand == 2) {
            } else if (!kBMN) {
              tma_load_2d_2cta(sB, &tmapB, bar, bk0 + kb * 64, nb0);           // box {64 k, 128 n}
            } else {
              tma_load_2d_2cta(sB, &tmapB, bar, nb0, bk0 + kb * 64);           // box {64 n, 64 k}
              tma_load_2d_2cta(sB + 8192, &tmapB, bar, nb0 + 64, bk0 + kb * 64);
            }
            if (kExpand) {
              const int f0 = kExpand == 1 ? m0 : nb0;                          // first feature of this CTA's half
              uint8_t* sP = pk_stage + stage * kPkStageBytes;
              mbar_arrive_expect_tx(&ctl->pk_full[stage], (uint32_t)kPkStageBytes);
              tma_load_2d(sP, &tmapPk, &ctl->pk_full[stage], f0 >> 1, kb * 64);          // values: box {64, 64}
              tma_load_2d(sP + 8192, &tmapMeta, &ctl->pk_full[stage], f0 >> 4, kb * 64); // metadata: box {8, 64}
            }
          } else {
            tma_load_2d_2cta(sA, &tmapA, bar, (ak0 >> 1) + kb * 64, m0);       // stored values: box {64, 128}
            // metadata atoms are rows of 2 x 1 KB in a [2 * atoms, 256] uint32 view (8-bit operands: a pair of
            // atoms per stage, 4 rows)
            const int atom = (m0 >> 7) * nkb_full + (ak0 >> 7) + kb;
            tma_load_2d_2cta(sM, &tmapMeta, bar, 0, (kFp8 ? 4 : 2) * atom);
            if (!kBMN) {
              tma_load_2d_2cta(sB, &tmapB, bar, bk0 + kb * 128, nb0);          // two 64-wide K slabs
              tma_load_2d_2cta(sB + kBSlabBytes, &tmapB, bar, bk0 + kb * 128 + 64, nb0);
            } else {
              tma_load_2d_2cta(sB, &tmapB, bar, nb0, bk0 + kb * 128);          // two chunks {64 n, 128 k}
              tma_load_2d_2cta(sB + 16384, &tmapB, bar, nb0 + 64, bk0 + kb * 128);
            }
          }
        }
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer (leader CTA only) ===========================
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = kFp8 ? idesc_e4m3(256, kBN, kSparse) : idesc_bf16(256, kBN, kAMN, kBMN, kSparse);
      // Descriptor halves that never change: high word = stride offset, version, swizzle; the low
      // word is (address >> 4) | leading offset, advanced by plain 32-bit adds.
      const uint32_t smem0 = smem_u32(smem);
      const uint64_t a_proto = (kMode == MODE_DENSE && kAMN) ? smem_desc(0, 8192, 1024, kSwizzle128B)
                                                             : smem_desc(0, 16, 1024, kSwizzle128B);
      const uint64_t b_proto = kBMN ? smem_desc(0, kSparse ? 16384 : 8192, 1024, kSwizzle128B)
                                    : smem_desc(0, 16, 1024, kSwizzle128B);
      const uint64_t m_proto = smem_desc(0, 128, 128, kSwizzleNone);
      const uint32_t a_hi = (uint32_t)(a_proto >> 32), b_hi = (uint32_t)(b_proto >> 32), m_hi = (uint32_t)(m_proto >> 32);
      const uint32_t a_lo0 = (uint32_t)a_proto + (smem0 >> 4);
      const uint32_t b_lo0 = (uint32_t)b_proto + ((smem0 + kAStageBytes) >> 4);
      const uint32_t m_lo0 = (uint32_t)m_proto + ((smem0 + kAStageBytes + kBHalfBytes) >> 4);
      // per-instruction advances of the low words (in 16-byte units)
      constexpr uint32_t a_step = (kMode == MODE_DENSE && kAMN) ? (2048 >> 4) : (32 >> 4);
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        const int nkb = args.tile_table ? __ldg(&args.tile_table[tile].nkb) : nkb_full;
        if (!mbar_wait(&ctl->tmem_empty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * kBN;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(&ctl->full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t soff = stage * (uint32_t)(kStageBytes >> 4);
          const uint32_t a_lo = a_lo0 + soff, b_lo = b_lo0 + soff;
          const uint32_t mbuf = tmem_base + kMetaCol + kMetaCols * ((uint32_t)kb & 1u);   // metadata double buffer
          if (kSparse) tmem_cp_128x128b_2cta(mbuf, desc64(m_lo0 + soff, m_hi));
          if (kSparse && kFp8) tmem_cp_128x128b_2cta(mbuf + 4u, desc64(m_lo0 + soff + (2048u >> 4), m_hi));
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t accum = (kb > 0 || k > 0) ? 1u : 0u;
            if (kSparse) {
              // K = 32 per instruction: 32 B of stored A, 64 B of B inside a 64-wide K slab
              const uint32_t bk = kBMN ? (uint32_t)k * (4096 >> 4)      // 32 k rows of 128 B
                                       : (uint32_t)((k >> 1) * (kBSlabBytes >> 4) + (k & 1) * (64 >> 4));
              if (kFp8)      // 64 logical K per instruction: two metadata columns each
                mma_sp_f8_2cta(tmem_d, desc64(a_lo + k * a_step, a_hi), desc64(b_lo + bk, b_hi), mbuf + 2u * (uint32_t)k,
                               idesc, accum);
              else
                mma_sp_f16_2cta(tmem_d, desc64(a_lo + k * a_step, a_hi), desc64(b_lo + bk, b_hi),
                                mbuf + (uint32_t)(k & ~1), idesc | (uint32_t)(k & 1), accum);
            } else {
              const uint32_t bk = (uint32_t)k * (kBMN ? (2048 >> 4) : (32 >> 4));
              if (kFp8) mma_f8_2cta(tmem_d, desc64(a_lo + k * a_step, a_hi), desc64(b_lo + bk, b_hi), idesc, accum);
              else      mma_f16_2cta(tmem_d, desc64(a_lo + k * a_step, a_hi), desc64(b_lo + bk, b_hi), idesc, accum);
            }
          }
          mma_commit_2cta(&ctl->empty[stage]);             // frees the stage in both CTAs
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        mma_commit_2cta(&ctl->tmem_full[acc]);             // accumulator ready, both CTAs
        if (++acc == (uint32_t)kAccBufs) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else if (kExpand != 0 && warp >= 6) {
    // =========================== operand expander (warps 6..13, both CTAs) ===========================
    // Stage tile = 64 tokens (K) x 128 features, MN-major, 128-byte swizzle: two chunks of 64 features,
    // a token row of a chunk is 128 bytes whose 16-byte units are XOR-ed with (token & 7). One unit is
    // eight features = two 2:4 groups = four stored values + one metadata byte in the packed tile.
    const int te = (int)threadIdx.x - 192;                 // 0..255
    const int seg = te & 15, tk0 = te >> 4;                // 16 units per token row; 16 tokens per pass
    const uint2* lut = ctl->expand_lut;
    uint32_t stage = 0, phase = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
      for (int kb = 0; kb < nkb_full; ++kb) {
        if (!mbar_wait(&ctl->pk_full[stage], phase, abort_flag)) { ok = false; break; }
        const uint8_t* sP = pk_stage + stage * kPkStageBytes;
        uint8_t* dst = smem + stage * kStageBytes + (kExpand == 1 ? 0 : kAStageBytes) + (seg >> 3) * 8192;
        uint2 v[4];
        uint32_t mb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int tk = tk0 + 16 * i;
          v[i] = *reinterpret_cast<const uint2*>(sP + tk * 128 + seg * 8);
          mb[i] = sP[8192 + tk * 16 + seg];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int tk = tk0 + 16 * i;
          const uint2 s0 = lut[mb[i] & 15u], s1 = lut[mb[i] >> 4];
          *reinterpret_cast<uint4*>(dst + tk * 128 + (((seg & 7) ^ (tk & 7)) << 4)) =
              make_uint4(__byte_perm(v[i].x, 0u, s0.x), __byte_perm(v[i].x, 0u, s0.y),
                         __byte_perm(v[i].y, 0u, s1.x), __byte_perm(v[i].y, 0u, s1.y));
        }
        // generic-proxy stores -> visible to the tensor core's async-proxy reads, then signal the stage
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive_leader(&ctl->full[stage]);
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if constexpr (kEpi == EPI_VNM8) {
    // =========================== fused activation epilogue (warps 2..9, both CTAs) ===========================
    // Two sets of four warps, one per accumulator buffer: set 0 takes this pair's even tiles, set 1 the odd
    // ones, so each set has two main loops' time for one tile.
    const int q = warp & 3, set = (warp - 2) >> 2;
    constexpr int kV = vnm_block(kBN);
    uint8_t* wsm = epi_stage + (set * 4 + q) * vnm_warp_bytes(kV);
    uint32_t acc_phase = 0;
    for (int tile = pair + set * num_pairs; tile < num_tiles; tile += 2 * num_pairs) {
      int mt, nt;
      tile_coords(tile, num_m_tiles, num_n_tiles_, mt, nt);
      const int64_t m0 = (int64_t)mt * 256 + (int64_t)rank * 128, n0 = (int64_t)nt * kBN;
      const uint32_t taddr = tmem_base + set * kBN + ((uint32_t)(q * 32) << 16);
      if (!mbar_wait(&ctl->tmem_full[set], acc_phase, abort_flag)) break;
      tc_fence_after();
      if (m0 >= args.M) {
        // M % 256 == 128: the second CTA of the last row of pairs holds no rows (its operand loads were
        // zero-filled); it only hands the accumulator back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_leader(&ctl->tmem_empty[set]);
      } else {
        // releases the accumulator itself, as soon as its last column has been read
        epi_vnm8_tile<kBN, kV>(args, taddr, m0, n0, args.N, q, lane, wsm, &ctl->tmem_empty[set]);
      }
      acc_phase ^= 1;
    }
  } else {
    // =========================== epilogue (warps 2..5, both CTAs) ===========================
    const int q = warp & 3;
    uint8_t* my_stage = epi_stage + q * 32 * kEpiStageRow;
    uint32_t acc = 0, acc_phase = 0;
    bool ok = true;
    for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
      const GemmTile tc = get_tile<kBN>(args, tile, num_m_tiles, num_n_tiles_, nkb_full);
      const int64_t m0 = (int64_t)tc.out_m + (int64_t)rank * 128, n0 = tc.out_n, n_limit = tc.n_limit;
      const uint32_t taddr = tmem_base + acc * kBN + ((uint32_t)(q * 32) << 16);
      uint4 ax[is_drelu_t(kEpi) ? kBN / 32 : 1][4];
      // M % 256 == 128 (regular raster only): the second CTA of the last row of pairs holds no rows
      const bool live = args.tile_table != nullptr || m0 < args.M;
      if (live) epi_prefetch<kEpi, kBN>(args, m0, n0, n_limit, q, lane, ax);
      if (!mbar_wait(&ctl->tmem_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      if (live) epi_tile<kEpi, kBN>(args, taddr, m0, n0, n_limit, q, lane, my_stage, ax);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&ctl->tmem_empty[acc]);
      if (++acc == (uint32_t)kAccBufs) { acc = 0; acc_phase ^= 1; }
    }
  }

  // =========================== teardown ===========================
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctl->abort_flag) atomicExch(args.status, 1);
  cluster_sync_all();                                    // the peer is done with our shared memory and barriers
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_2cta(tmem_base, kTmemCols);
  }
}

// ---- host side -----------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2D tensor map over a row-major [rows, cols] matrix of 2-byte (bf16, uint16) or 4-byte (uint32) elements;
// box = {box_cols, box_rows}.
int make_tmap(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
              uint32_t box_rows, CUtensorMapSwizzle swz, int kind = 0 /* 0 bf16, 1 uint32, 2 uint16 */) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return cuda_fail(cudaErrorUnknown);
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const bool u32 = kind == 1;
  cuuint64_t strides[1] = {(cuuint64_t)ld * (u32 ? 4 : 2)};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, u32 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : (kind == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), 2,
                  const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    g_last_cuda_error = (int)r;
    return SF_ERR_CUDA;
  }
  return SF_OK;
}

int sm_count() {
  static int n[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (n[dev] == 0) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n[dev] = v;
  }
  return n[dev];
}

template <int kMode, bool kAMN, bool kBMN, int kEpi>
int launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const GemmArgs& a, cudaStream_t s) {
  auto kern = gemm_tc_kernel<kMode, kAMN, kBMN, kEpi>;
  static bool attr_done[64] = {false};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_done[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(kMode != MODE_DENSE)));
    if (dev >= 0 && dev < 64) attr_done[dev] = true;
  }
  const int tiles = a.num_m_tiles * a.num_n_tiles;
  const int grid = tiles < sm_count() ? tiles : sm_count();
  kern<<<grid, kMode == MODE_VENOM ? kThreadsVenom : kThreads, smem_bytes(kMode != MODE_DENSE), s>>>(ta, tb, a);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

template <int kMode, bool kAMN, bool kBMN, int kEpi, int kBN = BN, int kExpand = 0, bool kFp8 = false>
int launch_two(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tm, GemmArgs a, cudaStream_t s,
               const CUtensorMap* tpk = nullptr) {
  auto kern = gemm_tc2_kernel<kMode, kAMN, kBMN, kEpi, kBN, kExpand, kFp8>;
  constexpr int smem = smem_bytes2(kMode != MODE_DENSE, kBN, kEpi, kExpand != 0, kFp8);
  static_assert(smem <= 232448, "shared memory per CTA");
  static bool attr_done[64] = {false};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_done[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    if (dev >= 0 && dev < 64) attr_done[dev] = true;
  }
  a.num_m_tiles = (int)((a.M + 255) / 256);
  a.num_n_tiles = (int)((a.N + kBN - 1) / kBN);
  // table-driven products: the table's length is on the device; launch for its upper bound
  const int tiles = a.tile_table ? a.num_k_blocks /* upper bound, see the grouped launchers */
                                 : a.num_m_tiles * a.num_n_tiles;
  const int max_pairs = sm_count() / 2;
  const int pairs = tiles < max_pairs ? tiles : max_pairs;
  kern<<<2 * pairs, threads2(kEpi, kExpand), smem, s>>>(ta, tb, tm, tpk ? *tpk : ta, a);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

// Tile width of the two-accumulator 2:4 variant (transposed-output products): 2 x 224 accumulator
// columns + 8 metadata columns fit the 512 TMEM columns.
#ifndef SF_NARROW_BN
#define SF_NARROW_BN 224
#endif
constexpr int kNarrowBN = SF_NARROW_BN;

// CTA pairs work on 256-row tiles; with M % 256 == 128 the second CTA of the last row of pairs runs on
// zero-filled operand rows and stores nothing. A single 128-row block runs the one-CTA kernels.
bool use_two_cta(int64_t M) { return M >= 256; }

}  // namespace

int make_tmap_2d(void* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                 uint32_t box_rows, bool swizzle128) {
  return make_tmap(reinterpret_cast<CUtensorMap*>(map), base, rows, cols, ld, box_cols, box_rows,
                   swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE);
}

int gemm_dense(const void* A, bool a_kmajor, const void* B, bool b_kmajor, int64_t M, int64_t N, int64_t K, int epi,
               void* C, int64_t ldc, void* C2, int64_t ldc2, const void* aux, int64_t ldaux, int* status,
               cudaStream_t s) {
  const bool two = use_two_cta(M);
  if (M % BM || N % (two ? 128 : BN) || K % 64) return SF_ERR_SHAPE;     // pairs: a ragged last tile of whole 32-column chunks
  if (M == 0 || N == 0) return SF_OK;
  CUtensorMap ta, tb;
  int st;
  if (a_kmajor) st = make_tmap(&ta, A, M, K, K, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  else          st = make_tmap(&ta, A, K, M, M, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  if (b_kmajor) st = make_tmap(&tb, B, N, K, K, 64, two ? 128 : 256, CU_TENSOR_MAP_SWIZZLE_128B);
  else          st = make_tmap(&tb, B, K, N, N, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K;
  a.C = C; a.ldc = ldc; a.C2 = C2; a.ldc2 = ldc2; a.aux = aux; a.ldaux = ldaux;
  a.status = status;
  a.num_m_tiles = (int)(M / BM); a.num_n_tiles = (int)(N / BN); a.num_k_blocks = (int)(K / 64);
#define SF_DENSE_CASE(AMN, BMN, EPI)                                              \
  return two ? launch_two<MODE_DENSE, AMN, BMN, EPI>(ta, tb, ta, a, s)            \
             : launch_one<MODE_DENSE, AMN, BMN, EPI>(ta, tb, a, s)
  const bool amn = !a_kmajor, bmn = !b_kmajor;
  if (epi == EPI_STORE) {
    if (!amn && !bmn) SF_DENSE_CASE(false, false, EPI_STORE);
    if (!amn && bmn) SF_DENSE_CASE(false, true, EPI_STORE);
    if (amn && !bmn) SF_DENSE_CASE(true, false, EPI_STORE);
    SF_DENSE_CASE(true, true, EPI_STORE);
  } else if (epi == EPI_SQRELU) {
    if (!amn && !bmn) SF_DENSE_CASE(false, false, EPI_SQRELU);
  } else if (epi == EPI_DRELU) {
    if (!amn && bmn) SF_DENSE_CASE(false, true, EPI_DRELU);
    if (!amn && !bmn) SF_DENSE_CASE(false, false, EPI_DRELU);
  }
#undef SF_DENSE_CASE
  return SF_ERR_UNSUPPORTED;
}

int gemm_sparse24(const void* a_vals, const uint8_t* meta_hw, const void* B, bool b_kmajor, int64_t M, int64_t N,
                  int64_t K, int epi, void* C, int64_t ldc, const void* aux, int64_t ldaux, int* status,
                  cudaStream_t s, const void* pack_meta, void* pack_vals) {
  if ((pack_meta != nullptr) != (pack_vals != nullptr) || (pack_vals && !is_drelu_t(epi))) return SF_ERR_UNSUPPORTED;
  const bool two = use_two_cta(M);
  if (epi == EPI_DRELU24_T && (!pack_vals || !aux || !two)) return SF_ERR_UNSUPPORTED;   // C (dense copy) optional
  if (M % BM || N % (two ? 128 : BN) || K % 128) return SF_ERR_SHAPE;
  if (M == 0 || N == 0) return SF_OK;
  const bool plain = (epi == EPI_STORE);                 // row-major output, either B layout: two-CTA kernel only
  if ((plain || !b_kmajor) && !two) return SF_ERR_UNSUPPORTED;
  CUtensorMap ta, tb, tm;
  int st = two ? make_tmap(&ta, a_vals, M, K / 2, K / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)
               : make_tmap(&ta, a_vals, M, K / 2, K / 2, 32, 128, CU_TENSOR_MAP_SWIZZLE_64B);
  if (st != SF_OK) return st;
  // transposed-output products on CTA pairs run 224-column tiles with two accumulators
  const bool narrow = two && !plain;
  if (b_kmajor) st = make_tmap(&tb, B, N, K, K, 64, two ? (narrow ? kNarrowBN / 2 : 128) : 256, CU_TENSOR_MAP_SWIZZLE_128B);
  else          st = make_tmap(&tb, B, K, N, N, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  tm = ta;
  if (two) {
    // hardware-ordered metadata: 2 KB atoms viewed as two rows of 256 uint32
    const int64_t atoms = (M / 128) * (K / 128);
    st = make_tmap(&tm, meta_hw, 2 * atoms, 256, 256, 256, 2, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
    if (st != SF_OK) return st;
  }
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K;
  a.C = C; a.ldc = ldc; a.aux = aux; a.ldaux = ldaux; a.meta_hw = meta_hw; a.status = status;
  a.pack_meta = pack_meta; a.pack_vals = pack_vals;
  a.num_m_tiles = (int)(M / BM); a.num_n_tiles = (int)(N / BN); a.num_k_blocks = (int)(K / 64);
  if (epi == EPI_STORE) {
    if (b_kmajor) return launch_two<MODE_SPARSE24, false, false, EPI_STORE>(ta, tb, tm, a, s);
    return launch_two<MODE_SPARSE24, false, true, EPI_STORE>(ta, tb, tm, a, s);
  }
  if (epi == EPI_STORE_T)
    return two ? launch_two<MODE_SPARSE24, false, false, EPI_STORE_T, kNarrowBN>(ta, tb, tm, a, s)
               : launch_one<MODE_SPARSE24, false, false, EPI_STORE_T>(ta, tb, a, s);
  if (epi == EPI_DRELU_T)
    return two ? launch_two<MODE_SPARSE24, false, false, EPI_DRELU_T, kNarrowBN>(ta, tb, tm, a, s)
               : launch_one<MODE_SPARSE24, false, false, EPI_DRELU_T>(ta, tb, a, s);
  if (epi == EPI_DRELU24_T) return launch_two<MODE_SPARSE24, false, false, EPI_DRELU24_T, kNarrowBN>(ta, tb, tm, a, s);
  return SF_ERR_UNSUPPORTED;
}

int gemm_route(const void* X, const void* means, int64_t T, int64_t D, int E, int* expert, float* logits, int* status,
               cudaStream_t s) {
  if (T % 256 || D % 64 || E < 1 || E > 16) return SF_ERR_SHAPE;
  if (T == 0) return SF_OK;
  CUtensorMap ta, tb;
  int st = make_tmap(&ta, X, T, D, D, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, means, E, D, D, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);     // rows beyond E arrive as zeros
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = T; a.N = 256; a.K = D;
  a.status = status;
  a.route_expert = expert; a.route_logits = logits; a.route_E = E;
  a.num_k_blocks = (int)(D / 64);
  return launch_two<MODE_DENSE, false, false, EPI_ROUTE>(ta, tb, ta, a, s);
}

int gemm_fp8(bool sparse, const void* A, const uint8_t* meta_hw, const void* B, int64_t M, int64_t N, int64_t K,
             float alpha, void* C, int64_t ldc, int* status, cudaStream_t s) {
  if (M % 256 || N % 32 || K % (sparse ? 256 : 128) || (sparse && !meta_hw)) return SF_ERR_SHAPE;
  if (M == 0 || N == 0) return SF_OK;
  // the operands in 2-byte units: [M, K/2] (dense) or [M, K/4] (2:4 values), [N, K/2]
  const int64_t K2 = K / 2;
  CUtensorMap ta, tb, tm;
  int st = sparse ? make_tmap(&ta, A, M, K2 / 2, K2 / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B, 2)
                  : make_tmap(&ta, A, M, K2, K2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B, 2);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, B, N, K2, K2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B, 2);
  if (st != SF_OK) return st;
  tm = ta;
  if (sparse) {
    // per 128 rows and 256 logical K: two 2 KB atoms = four rows of the [4 * atom pairs, 256] uint32 view
    const int64_t pairs = (M / 128) * (K / 256);
    st = make_tmap(&tm, meta_hw, 4 * pairs, 256, 256, 256, 4, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
    if (st != SF_OK) return st;
  }
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K2;
  a.C = C; a.ldc = ldc; a.meta_hw = meta_hw; a.status = status; a.out_scale = alpha;
  a.num_k_blocks = (int)(K2 / 64);
  if (sparse) return launch_two<MODE_SPARSE24, false, false, EPI_STORE, BN, 0, true>(ta, tb, tm, a, s);
  return launch_two<MODE_DENSE, false, false, EPI_STORE, BN, 0, true>(ta, tb, tm, a, s);
}

bool gemm_sparse24_vnm8_supported(int64_t F, int64_t T, int64_t D, int V) {
  return F >= 256 && T > 0 && F % 128 == 0 && D % 128 == 0 && (V == 64 || V == 128) && T % V == 0;
}

int gemm_sparse24_vnm8(const void* a_vals, const uint8_t* meta_hw, const void* X, int64_t F, int64_t T, int64_t D,
                       int V, const Vnm8Out& out, int* status, cudaStream_t s) {
  if (!gemm_sparse24_vnm8_supported(F, T, D, V)) return SF_ERR_SHAPE;
  // Token tiles hold whole V-blocks: three blocks of 64 (192 columns) or one block of 128.
  const int bn = V == 64 ? 192 : 128;
  CUtensorMap ta, tb, tm;
  int st = make_tmap(&ta, a_vals, F, D / 2, D / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, X, T, D, D, 64, bn / 2, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  const int64_t atoms = (F / 128) * (D / 128);
  st = make_tmap(&tm, meta_hw, 2 * atoms, 256, 256, 256, 2, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = F; a.N = T; a.K = D; a.V = V;
  a.meta_hw = meta_hw; a.status = status;
  a.vn_vals = out.vals; a.vn_relu = out.relu; a.vn_meta = out.meta; a.vn_colidx = out.colidx;
  a.vn_vals24 = out.vals24; a.vn_relu24 = out.relu24; a.vn_meta24 = out.meta24; a.vn_meta24_hw = out.meta24_hw;
  a.vn_y1 = out.y1; a.vn_dense = out.dense;
  if (V == 64) return launch_two<MODE_SPARSE24, false, false, EPI_VNM8, 192>(ta, tb, tm, a, s);
  return launch_two<MODE_SPARSE24, false, false, EPI_VNM8, 128>(ta, tb, tm, a, s);
}

// ---- grouped (table-driven) products of the routed step --------------------------------------------------
// All of them run on CTA pairs; the caller's tables hold one entry per output tile and `max_tiles` bounds
// their length (it sizes the grid; GemmArgs::num_k_blocks carries it to the launcher).

int gemm_grouped_act24(const void* a_vals, const uint8_t* meta_hw, const void* Xp, int64_t rows, int64_t F, int64_t Fe,
                       int64_t D, const Act24Out& out, const GemmTile* tiles, const int* num_tiles, int max_tiles,
                       int* status, cudaStream_t s) {
  if (F % 256 || Fe % 256 || D % 128 || rows % 32 || max_tiles <= 0) return SF_ERR_SHAPE;
  CUtensorMap ta, tb, tm;
  int st = make_tmap(&ta, a_vals, F, D / 2, D / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, Xp, rows, D, D, 64, kNarrowBN / 2, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tm, meta_hw, 2 * (F / 128) * (D / 128), 256, 256, 256, 2, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = Fe; a.N = rows; a.K = D;                           // M: width of the outputs (features per expert)
  a.status = status;
  a.vn_vals24 = out.vals; a.vn_relu24 = out.relu; a.vn_meta24 = out.meta; a.vn_meta24_hw = out.meta_hw;
  a.vn_dense = out.dense; a.vn_y1 = out.y1;
  a.tile_table = tiles; a.num_tiles_dev = num_tiles; a.num_k_blocks = max_tiles;
  return launch_two<MODE_SPARSE24, false, false, EPI_ACT24_T, kNarrowBN>(ta, tb, tm, a, s);
}

int gemm_grouped_drelu24(const void* a_vals, const uint8_t* meta_hw, const void* dYp, int64_t rows, int64_t F,
                         int64_t Fe, int64_t D, const void* relu_vals, const void* meta, void* pack_vals, void* dense,
                         const GemmTile* tiles, const int* num_tiles, int max_tiles, int* status, cudaStream_t s) {
  if (F % 256 || Fe % 256 || D % 128 || rows % 32 || max_tiles <= 0) return SF_ERR_SHAPE;
  CUtensorMap ta, tb, tm;
  int st = make_tmap(&ta, a_vals, F, D / 2, D / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, dYp, rows, D, D, 64, kNarrowBN / 2, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tm, meta_hw, 2 * (F / 128) * (D / 128), 256, 256, 256, 2, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = Fe; a.N = rows; a.K = D;
  a.C = dense; a.ldc = Fe; a.aux = relu_vals; a.pack_meta = meta; a.pack_vals = pack_vals;
  a.status = status;
  a.tile_table = tiles; a.num_tiles_dev = num_tiles; a.num_k_blocks = max_tiles;
  return launch_two<MODE_SPARSE24, false, false, EPI_DRELU24_T, kNarrowBN>(ta, tb, tm, a, s);
}

int gemm_grouped_sparse24_rm(const void* a_vals, const uint8_t* meta_hw, const void* B, bool b_kmajor, int64_t rows,
                             int64_t N, int64_t Fe, int64_t Ktot, void* C, const int* row_map, const GemmTile* tiles,
                             const int* num_tiles, int max_tiles, int* status, cudaStream_t s) {
  if (rows % 256 || N % 256 || Fe % 128 || Ktot % Fe || max_tiles <= 0) return SF_ERR_SHAPE;
  CUtensorMap ta, tb, tm;
  int st = make_tmap(&ta, a_vals, rows, Fe / 2, Fe / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  if (b_kmajor) st = make_tmap(&tb, B, N, Ktot, Ktot, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  else          st = make_tmap(&tb, B, Ktot, N, N, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tm, meta_hw, 2 * (rows / 128) * (Fe / 128), 256, 256, 256, 2, CU_TENSOR_MAP_SWIZZLE_NONE, 1);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = rows; a.N = N; a.K = Fe;                           // K of the packed operand: its metadata atoms follow it
  a.C = C; a.ldc = N; a.status = status; a.row_map = row_map;
  a.tile_table = tiles; a.num_tiles_dev = num_tiles; a.num_k_blocks = max_tiles;
  if (b_kmajor) return launch_two<MODE_SPARSE24, false, false, EPI_STORE>(ta, tb, tm, a, s);
  return launch_two<MODE_SPARSE24, false, true, EPI_STORE>(ta, tb, tm, a, s);
}

int gemm_grouped_dense_tn(const void* A, int64_t Ma, const void* B, int64_t Nb, int64_t rows, void* C, int64_t ldc,
                          const GemmTile* tiles, const int* num_tiles, int max_tiles, int* status, cudaStream_t s) {
  if (Ma % 256 || Nb % 256 || rows % 64 || max_tiles <= 0) return SF_ERR_SHAPE;
  CUtensorMap ta, tb;
  int st = make_tmap(&ta, A, rows, Ma, Ma, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, B, rows, Nb, Nb, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = Ma; a.N = ldc; a.K = rows;                         // N bounds the stored columns: the whole output row
  a.C = C; a.ldc = ldc; a.status = status;
  a.tile_table = tiles; a.num_tiles_dev = num_tiles; a.num_k_blocks = max_tiles;
  return launch_two<MODE_DENSE, true, true, EPI_STORE>(ta, tb, ta, a, s);
}

int gemm_dense_expand(const void* dense_op, int packed_operand, const void* pk_vals, const void* pk_meta, int64_t M,
                      int64_t N, int64_t K, void* C, int64_t ldc, int* status, cudaStream_t s) {
  if (M % 256 || N % 256 || K % 64 || (packed_operand != 1 && packed_operand != 2)) return SF_ERR_SHAPE;
  if (M == 0 || N == 0) return SF_OK;
  const int64_t X = packed_operand == 1 ? M : N;                              // width of the packed operand
  CUtensorMap ta, tb, tm, tp;
  // the dense operand: [K, M] or [K, N] row-major, 64 x 64 boxes
  int st = make_tmap(packed_operand == 1 ? &tb : &ta, dense_op, K, packed_operand == 1 ? N : M,
                     packed_operand == 1 ? N : M, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
  if (st != SF_OK) return st;
  if (packed_operand == 1) ta = tb; else tb = ta;                             // the unused map only has to be valid
  st = make_tmap(&tp, pk_vals, K, X / 2, X / 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_NONE);
  if (st != SF_OK) return st;
  st = make_tmap(&tm, pk_meta, K, X / 16, X / 16, 8, 64, CU_TENSOR_MAP_SWIZZLE_NONE, 2);
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K;
  a.C = C; a.ldc = ldc; a.status = status;
  a.num_m_tiles = (int)(M / BM); a.num_n_tiles = (int)(N / BN); a.num_k_blocks = (int)(K / 64);
  if (packed_operand == 1) return launch_two<MODE_DENSE, true, true, EPI_STORE, BN, 1>(ta, tb, tm, a, s, &tp);
  return launch_two<MODE_DENSE, true, true, EPI_STORE, BN, 2>(ta, tb, tm, a, s, &tp);
}

int gemm_venom(const void* a_vals, const uint8_t* meta_hw, const uint8_t* colidx, const void* Bt, int64_t T,
               int64_t F, int64_t N, int V, int Mv, void* C, int64_t ldc, int* status, cudaStream_t s) {
  const int64_t Kc = 4 * F / Mv;                                               // condensed reduction length
  if (T % BM || N % BN || Kc % 128 || (V != 64 && V != 128)) return SF_ERR_SHAPE;
  if (T == 0 || N == 0) return SF_OK;
  CUtensorMap ta, tb;
  int st = make_tmap(&ta, a_vals, T, Kc / 2, Kc / 2, 32, V == 64 ? 64 : 128, CU_TENSOR_MAP_SWIZZLE_64B);
  if (st != SF_OK) return st;
  st = make_tmap(&tb, Bt, F, N, N, 64, 1, CU_TENSOR_MAP_SWIZZLE_128B);        // row gather: one row per box
  if (st != SF_OK) return st;
  GemmArgs a{};
  a.gather_tma_groups = 12;      // measured optimum of the TMA : cp.async split (of 16 groups per stage)
  a.M = T; a.N = N; a.K = Kc;
  a.aux = Bt; a.ldaux = N;
  a.C = C; a.ldc = ldc; a.meta_hw = meta_hw; a.colidx = colidx; a.V = V; a.Mv = Mv; a.G = F / Mv;
  a.status = status;
  a.num_m_tiles = (int)(T / BM); a.num_n_tiles = (int)(N / BN); a.num_k_blocks = (int)(Kc / 64);
  return launch_one<MODE_VENOM, false, true, EPI_STORE>(ta, tb, a, s);
}

}  // namespace sf
