// SquaredReLU + V:N:M (Venom) activation sparsification (Eq. 2, Section 2.3, Table 5).
//
// One CTA owns a strip of V rows x kCW columns (kCW / M blocks of V x M). The strip is staged in
// shared memory once, so every input element is read from HBM exactly once:
//   pass A  one thread per column: float32 score = sum over the V rows, first to last, of the
//           magnitude of the stored activation; the four best columns of each M-column group
//           stay (ties to the lower index) and are recorded in ascending order;
//   pass B  one thread per (row, group): 2:4 among the four kept columns, emit two values, the
//           two matching ReLU values, one metadata nibble (four neighbours form a uint16).
// The accumulation order of pass A is part of the format: it is what makes the mask unique.
#include "sf_common.cuh"
#include "sparse_fmt.cuh"

namespace sf {

namespace {

constexpr int kCW = 256;          // columns per CTA strip (>= 4 groups of the widest M)
constexpr int kPad = 8;           // 16 B row padding (bank spread)
constexpr int kThreads = 256;
static_assert(kThreads >= kCW && kThreads % (kCW / 8) == 0, "one thread per strip column in the ranking steps");

__device__ __forceinline__ void sqrelu_bits(uint32_t x, bool apply, uint32_t& h, uint32_t& relu) {
  if (!apply) { h = x; relu = 0; return; }
  const float y = bf16_bits_to_float(x);
  const float r = y > 0.f ? y : 0.f;
  relu = y > 0.f ? x : 0u;
  h = float_to_bf16_bits(__fmul_rn(r, r));
}

// One group of M columns of a dense row: values va, vb at columns ca < cb, +0 elsewhere.
__device__ __forceinline__ void write_group_dense(uint16_t* drow, int M, uint32_t ca, uint32_t cb, uint32_t va,
                                                  uint32_t vb) {
  for (int m8 = 0; m8 < M; m8 += 8) {
    uint32_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t col = (uint32_t)(m8 + e);
      const uint32_t val = (col == ca) ? va : (col == cb) ? vb : 0u;
      const uint32_t sh = val << (16 * (e & 1));
      if (e < 2) w0 |= sh; else if (e < 4) w1 |= sh; else if (e < 6) w2 |= sh; else w3 |= sh;
    }
    if (M >= 8) {
      *reinterpret_cast<uint4*>(drow + m8) = make_uint4(w0, w1, w2, w3);
    } else {                                              // M == 4: one 8-byte group
      *reinterpret_cast<uint2*>(drow) = make_uint2(w0, w1);
    }
  }
}

__device__ __forceinline__ uint32_t relu2(uint32_t w) { return bf2_relu(w); }
__device__ __forceinline__ uint32_t sq2(uint32_t r) { return bf2_sq(r); }

// kW: strip width in columns (128 for M <= 32: half the shared memory, twice the resident CTAs; 256 for M = 64).
template <int kW>
__global__ void __launch_bounds__(kThreads)
vnm_kernel(const uint16_t* __restrict__ P, int64_t T, int64_t F, int64_t ld, int V, int M, int apply,
           uint16_t* __restrict__ vals, uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw,
           uint8_t* __restrict__ colidx, uint16_t* __restrict__ relu_vals, uint16_t* __restrict__ dense_out,
           uint16_t* __restrict__ relu_dense_out) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint16_t* tile = reinterpret_cast<uint16_t*>(smem_raw);                        // [V][kW + kPad]
  uint32_t* score = reinterpret_cast<uint32_t*>(tile + (size_t)V * (kW + kPad)); // [kW] float bits
  uint8_t* keepf = reinterpret_cast<uint8_t*>(score + kW);                       // [kW]
  uint8_t* cidx = keepf + kW;                                                    // [kW / 4][4]
  constexpr int kRow = kW + kPad;

  const int tid = threadIdx.x;
  const int64_t c0 = (int64_t)blockIdx.x * kW;
  const int64_t blk = blockIdx.y;
  const int64_t t0 = blk * V;
  const int cvalid = (int)min((int64_t)kW, F - c0);
  const int64_t G = F / M;

  // ---- stage the strip
  for (int i = tid; i < V * (kW / 8); i += kThreads) {
    const int r = i / (kW / 8), cc = (i % (kW / 8)) * 8;
    if (cc < cvalid) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(P + (t0 + r) * ld + c0 + cc));
      *reinterpret_cast<uint4*>(tile + r * kRow + cc) = q;
    }
  }
  __syncthreads();

  // ---- pass A: column scores (sequential float32 adds, rows in ascending order), two columns per
  // thread on packed bf16 pairs: max with zero, then one correctly rounded bf16 multiply (equal to
  // rounding the exact float32 square)
  if (tid < kW / 2) {
    float s0 = 0.f, s1 = 0.f;
    if (2 * tid < cvalid) {
      const uint32_t* col = reinterpret_cast<const uint32_t*>(tile) + tid;
      // eight rows per trip: the loads and the packed arithmetic of a trip are independent, only the
      // two add chains are sequential; a tail loop takes V % 8 rows
      int r = 0;
      for (; r + 8 <= V; r += 8) {
        uint32_t h[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t w = col[(r + u) * (kRow / 2)];
          h[u] = apply ? sq2(relu2(w)) : (w & 0x7FFF7FFFu);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          s0 = __fadd_rn(s0, __uint_as_float(h[u] << 16));
          s1 = __fadd_rn(s1, __uint_as_float(h[u] & 0xFFFF0000u));
        }
      }
      for (; r < V; ++r) {
        const uint32_t w = col[r * (kRow / 2)];
        const uint32_t h = apply ? sq2(relu2(w)) : (w & 0x7FFF7FFFu);
        s0 = __fadd_rn(s0, __uint_as_float(h << 16));
        s1 = __fadd_rn(s1, __uint_as_float(h & 0xFFFF0000u));
      }
    }
    score[2 * tid] = __float_as_uint(s0);
    score[2 * tid + 1] = __float_as_uint(s1);
  }
  __syncthreads();
  if (tid < kW) {
    const int j = tid, jm = j % M, base = j - jm;
    const uint32_t s = score[j];
    int rank = 0;
    for (int i = 0; i < M; ++i) {
      const uint32_t si = score[base + i];
      rank += (si > s) || (si == s && i < jm);
    }
    keepf[j] = rank < 4;
  }
  __syncthreads();
  if (tid < kW) {
    const int j = tid, jm = j % M, base = j - jm;
    if (keepf[j] && j < cvalid) {
      int pos = 0;
      for (int i = 0; i < jm; ++i) pos += keepf[base + i];
      cidx[(j / M) * 4 + pos] = (uint8_t)jm;
    }
  }
  __syncthreads();
  const int ng = cvalid / M;                                  // groups in this strip (multiple of 4)
  if (tid < ng) {
    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + tid * 4);
    *reinterpret_cast<uint32_t*>(colidx + (blk * G + c0 / M + tid) * 4) = c4;
  }

  // ---- pass B: 2:4 inside the kept columns
  const int64_t g0 = c0 / M;
  const int rstep_fast = ng > 0 ? kThreads / ng : 0;
  if (ng > 0 && kThreads % ng == 0 && (32 % ng == 0 || ng % 32 == 0) && V % rstep_fast == 0) {
    // Fast form: a thread always serves group tid % ng, for rows tid / ng, tid / ng + kThreads / ng, ...;
    // the four kept columns, hence the four shared-memory offsets, are fixed per thread. Packed bf16
    // arithmetic on the four kept values only; the ReLU pair reuses the byte-permute selector of the
    // value pair; the dense copies are built in registers and written with whole 16-byte stores.
    const int g = tid % ng, rstep = rstep_fast, r0 = tid / ng;
    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + g * 4);
    const uint16_t* tp = tile + r0 * kRow + g * M;
    const int o0 = (int)(c4 & 0xFFu), o1 = (int)((c4 >> 8) & 0xFFu), o2 = (int)((c4 >> 16) & 0xFFu), o3 = (int)(c4 >> 24);
    const bool lead4 = (g & 3) == 0;
    const bool want_relu = relu_vals && apply;
    const int64_t trow = t0 + r0;
    uint16_t* p_vals = vals + trow * (2 * G) + 2 * (g0 + g);
    uint16_t* p_relu = want_relu ? relu_vals + trow * (2 * G) + 2 * (g0 + g) : nullptr;
    uint16_t* p_dense = dense_out ? dense_out + trow * F + c0 + g * M : nullptr;
    uint16_t* p_rdense = relu_dense_out ? relu_dense_out + trow * F + c0 + g * M : nullptr;
    uint16_t* p_meta = meta + trow * (G >> 2) + ((g0 + g) >> 2);
    const int64_t kw = (g0 + g) >> 2;
    const int64_t s_vals = (int64_t)rstep * (2 * G), s_dense = (int64_t)rstep * F, s_meta = (int64_t)rstep * (G >> 2);
    for (int r = r0; r < V; r += rstep) {
      const uint32_t lo = (uint32_t)tp[o0] | ((uint32_t)tp[o1] << 16), hi = (uint32_t)tp[o2] | ((uint32_t)tp[o3] << 16);
      const uint32_t rl_lo = apply ? relu2(lo) : 0u, rl_hi = apply ? relu2(hi) : 0u;
      const uint32_t h_lo = apply ? sq2(rl_lo) : lo, h_hi = apply ? sq2(rl_hi) : hi;
      uint32_t packed;
      const uint32_t nib = top2of4_packed(h_lo, h_hi, &packed);
      const uint32_t p0 = nib & 3u, p1 = nib >> 2;
      *reinterpret_cast<uint32_t*>(p_vals) = packed;
      const uint32_t rpair = __byte_perm(rl_lo, rl_hi, 0x1010u + p0 * 0x22u + p1 * 0x2200u);
      if (want_relu) *reinterpret_cast<uint32_t*>(p_relu) = rpair;
      if (dense_out || relu_dense_out) {
        // whole 16-byte stores only: word j of the group holds the value kept at column 2j or 2j + 1
        const uint32_t ca = (c4 >> (8 * p0)) & 0xFFu, cb = (c4 >> (8 * p1)) & 0xFFu;       // kept columns, ca < cb
        const uint32_t wa = ca >> 1, wb = cb >> 1, sa = 16u * (ca & 1u), sb = 16u * (cb & 1u);
        const uint32_t ha = (packed & 0xFFFFu) << sa, hb = (packed >> 16) << sb;
        const uint32_t ra = (rpair & 0xFFFFu) << sa, rb = (rpair >> 16) << sb;
        if (M >= 8) {
          for (int m8 = 0; m8 < M; m8 += 8) {
            uint32_t dw[4], rw4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t wj = (uint32_t)(m8 >> 1) + j;
              const bool ia = wa == wj, ib = wb == wj;
              dw[j] = (ia ? ha : 0u) | (ib ? hb : 0u);
              rw4[j] = (ia ? ra : 0u) | (ib ? rb : 0u);
            }
            if (dense_out) *reinterpret_cast<uint4*>(p_dense + m8) = make_uint4(dw[0], dw[1], dw[2], dw[3]);
            if (relu_dense_out) *reinterpret_cast<uint4*>(p_rdense + m8) = make_uint4(rw4[0], rw4[1], rw4[2], rw4[3]);
          }
        } else {                                            // M == 4: one 8-byte group
          const uint32_t d0 = (wa == 0u ? ha : 0u) | (wb == 0u ? hb : 0u), d1 = (wa == 1u ? ha : 0u) | (wb == 1u ? hb : 0u);
          const uint32_t q0 = (wa == 0u ? ra : 0u) | (wb == 0u ? rb : 0u), q1 = (wa == 1u ? ra : 0u) | (wb == 1u ? rb : 0u);
          if (dense_out) *reinterpret_cast<uint2*>(p_dense) = make_uint2(d0, d1);
          if (relu_dense_out) *reinterpret_cast<uint2*>(p_rdense) = make_uint2(q0, q1);
        }
      }
      uint32_t word = nib;
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 4;
      word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 8;
      if (lead4) {
        *p_meta = (uint16_t)word;
        if (meta_hw) *reinterpret_cast<uint16_t*>(meta_hw + meta_hw_offset(t0 + r, kw, 4 * G)) = (uint16_t)word;
      }
      tp += rstep * kRow;
      p_vals += s_vals;
      if (want_relu) p_relu += s_vals;
      if (dense_out) p_dense += s_dense;
      if (relu_dense_out) p_rdense += s_dense;
      p_meta += s_meta;
    }
    return;
  }
  // General form (ragged strips, V not a multiple of the row step): one (row, group) item per thread
  const int items = V * ng;
  const int items_pad = (items + 31) & ~31;
  for (int i = tid; i < items_pad; i += kThreads) {
    const bool valid = i < items;
    const int r = valid ? i / ng : 0, g = valid ? i - r * ng : 0;
    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + g * 4);
    const uint16_t* row = tile + r * kRow + g * M;
    uint32_t h[4], rl[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) sqrelu_bits(row[(c4 >> (8 * k)) & 0xFFu], apply, h[k], rl[k]);
    const uint32_t nib = top2of4(h[0] & 0x7FFFu, h[1] & 0x7FFFu, h[2] & 0x7FFFu, h[3] & 0x7FFFu);
    const uint32_t p0 = nib & 3u, p1 = nib >> 2;
    const uint32_t v0 = p0 == 0 ? h[0] : p0 == 1 ? h[1] : h[2];
    const uint32_t v1 = p1 == 1 ? h[1] : p1 == 2 ? h[2] : h[3];
    const int64_t t = t0 + r;
    if (valid) {
      *reinterpret_cast<uint32_t*>(vals + t * (2 * G) + 2 * (g0 + g)) = v0 | (v1 << 16);
      const uint32_t r0 = p0 == 0 ? rl[0] : p0 == 1 ? rl[1] : rl[2];
      const uint32_t r1 = p1 == 1 ? rl[1] : p1 == 2 ? rl[2] : rl[3];
      if (relu_vals && apply) *reinterpret_cast<uint32_t*>(relu_vals + t * (2 * G) + 2 * (g0 + g)) = r0 | (r1 << 16);
      const uint32_t ca = (c4 >> (8 * p0)) & 0xFFu, cb = (c4 >> (8 * p1)) & 0xFFu;
      if (dense_out) write_group_dense(dense_out + t * F + c0 + g * M, M, ca, cb, v0, v1);
      if (relu_dense_out) write_group_dense(relu_dense_out + t * F + c0 + g * M, M, ca, cb, r0, r1);
    }
    // four neighbouring groups of a row -> one metadata word (ng is a multiple of 4)
    uint32_t word = valid ? nib : 0u;
    word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 4;
    word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 8;
    if (valid && (g & 3) == 0) {
      const int64_t kw = (g0 + g) >> 2;
      meta[t * (G >> 2) + kw] = (uint16_t)word;
      if (meta_hw) *reinterpret_cast<uint16_t*>(meta_hw + meta_hw_offset(t, kw, 4 * G)) = (uint16_t)word;
    }
  }
}


// ---- M = 8 fast path ---------------------------------------------------------------------------
// Same computation as vnm_kernel for groups of eight columns, written for a low instruction count:
// packed bf16x2 arithmetic (max with zero, then one correctly rounded bf16 multiply, which equals
// rounding the exact float32 square), whole 16-byte groups from shared memory, byte permutes with
// selectors that depend only on the block's kept columns (constant per thread: a thread always
// serves the same group of the strip), and mask words for the dense copies.
template <int kW>
__global__ void __launch_bounds__(kThreads)
vnm8_kernel(const uint16_t* __restrict__ P, int64_t T, int64_t F, int64_t ld, int V, int apply,
            uint16_t* __restrict__ vals, uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw,
            uint8_t* __restrict__ colidx, uint16_t* __restrict__ relu_vals, uint16_t* __restrict__ dense_out,
            uint16_t* __restrict__ relu_dense_out, uint16_t* __restrict__ vals24, uint16_t* __restrict__ meta24,
            uint8_t* __restrict__ meta24_hw, uint16_t* __restrict__ relu24) {
  constexpr int M = 8;
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint16_t* tile = reinterpret_cast<uint16_t*>(smem_raw);                        // [V][kW + kPad]
  uint32_t* score = reinterpret_cast<uint32_t*>(tile + (size_t)V * (kW + kPad));
  uint8_t* keepf = reinterpret_cast<uint8_t*>(score + kW);
  uint8_t* cidx = keepf + kW;
  uint4* sel_tab = reinterpret_cast<uint4*>(cidx + kW);                          // [kW / 8][7] selector words
  uint8_t* nib_tab = reinterpret_cast<uint8_t*>(sel_tab + (kW / 8) * 7);         // [kW / 8][7] 2:4-view nibble pairs
  constexpr int kRow = kW + kPad;

  const int tid = threadIdx.x;
  const int64_t c0 = (int64_t)blockIdx.x * kW;
  const int64_t blk = blockIdx.y;
  const int64_t t0 = blk * V;
  const int cvalid = (int)min((int64_t)kW, F - c0);
  const int64_t G = F / M;

  for (int i = tid; i < V * (kW / 8); i += kThreads) {
    const int r = i / (kW / 8), cc = (i % (kW / 8)) * 8;
    if (cc < cvalid) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(P + (t0 + r) * ld + c0 + cc));
      *reinterpret_cast<uint4*>(tile + r * kRow + cc) = q;
    }
  }
  __syncthreads();

  // pass A: two columns per thread, rows first to last, one float32 add per element
  if (tid < kW / 2) {
    float s0 = 0.f, s1 = 0.f;
    if (2 * tid < cvalid) {
      const uint32_t* col = reinterpret_cast<const uint32_t*>(tile) + tid;
      // eight rows per trip (V is a multiple of 8): the loads and the packed arithmetic of a trip are
      // independent, only the two add chains are sequential
      for (int r = 0; r < V; r += 8) {
        uint32_t h[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t w = col[(r + u) * (kRow / 2)];
          h[u] = apply ? sq2(relu2(w)) : (w & 0x7FFF7FFFu);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          s0 = __fadd_rn(s0, __uint_as_float(h[u] << 16));
          s1 = __fadd_rn(s1, __uint_as_float(h[u] & 0xFFFF0000u));
        }
      }
    }
    score[2 * tid] = __float_as_uint(s0);
    score[2 * tid + 1] = __float_as_uint(s1);
  }
  __syncthreads();
  if (tid < kW) {
    const int j = tid, jm = j & 7, base = j - jm;
    const uint32_t s = score[j];
    int rank = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) {
      const uint32_t si = score[base + i];
      rank += (si > s) || (si == s && i < jm);
    }
    keepf[j] = rank < 4;
  }
  __syncthreads();
  if (tid < kW) {
    const int j = tid, jm = j & 7, base = j - jm;
    if (keepf[j] && j < cvalid) {
      int pos = 0;
      for (int i = 0; i < jm; ++i) pos += keepf[base + i];
      cidx[(j >> 3) * 4 + pos] = (uint8_t)jm;
    }
  }
  __syncthreads();
  const int ng = cvalid / M;                                  // multiple of 4; kThreads % ng == 0
  if (tid < ng) {
    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + tid * 4);
    *reinterpret_cast<uint32_t*>(colidx + (blk * G + c0 / M + tid) * 4) = c4;
  }

  // Selector table: a group's row keeps one of six position pairs (i < j) of its four kept columns.
  // Everything the row loop derives from that pair -- byte-permute selectors that scatter the two
  // kept values into the four dense words, pick the two ReLU values out of the row's words, and lay
  // the pair out as a plain 2:4 operand with its nibble pair -- depends on (group, pair) only, so
  // it is tabulated once per strip: slot = nibble % 7 is distinct for the six legal nibbles.
  if (tid < ng * 6) {
    const int ge = tid / 6, pe = tid - ge * 6;
    const int pi = pe < 3 ? 0 : (pe < 5 ? 1 : 2), pj = pe < 3 ? pe + 1 : (pe < 5 ? pe - 1 : 3);
    const uint32_t ca = cidx[ge * 4 + pi], cb = cidx[ge * 4 + pj];                // kept columns, ca < cb
    const uint32_t nibp = (uint32_t)pi | ((uint32_t)pj << 2);
    uint4 selv;
    uint32_t nib24;
    vnm8_pair_selectors(ca, cb, selv, nib24);
    const int slot = ge * 7 + (int)(nibp % 7u);
    sel_tab[slot] = selv;
    nib_tab[slot] = (uint8_t)nib24;
  }
  __syncthreads();

  // pass B: a thread serves one group g = tid % ng for rows tid / ng, tid / ng + kThreads / ng, ...
  // Everything that depends only on (thread, group) is computed once; the row loop advances
  // pointers by constant strides.
  const int g = tid % ng, rstep = kThreads / ng, r0 = tid / ng;
  const int64_t g0 = c0 / M;
  const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + g * 4);
  uint32_t selp[2], mhi[2];
#pragma unroll
  for (int pr = 0; pr < 2; ++pr) {
    const uint32_t ca = (c4 >> (16 * pr)) & 0xFFu, cb = (c4 >> (16 * pr + 8)) & 0xFFu;
    const uint32_t sa = 2u * (ca & 3u), sb = 2u * (cb & 3u);
    selp[pr] = sa | ((sa + 1u) << 4) | (sb << 8) | ((sb + 1u) << 12);
    mhi[pr] = ((ca & 4u) ? 0x0000FFFFu : 0u) | ((cb & 4u) ? 0xFFFF0000u : 0u);   // take from columns 4..7
  }
  const bool lead4 = (g & 3) == 0, lead2 = (g & 1) == 0;
  const bool want_relu = relu_vals && apply, want24 = vals24 != nullptr;
  const bool need_relu_pair = want_relu || (relu_dense_out != nullptr) || (relu24 != nullptr && apply);
  const int64_t trow = t0 + r0;
  const uint16_t* tp = tile + r0 * kRow + g * M;
  const uint4* my_sel = sel_tab + g * 7;
  const uint8_t* my_nib = nib_tab + g * 7;
  uint16_t* p_vals = vals + trow * (2 * G) + 2 * (g0 + g);
  uint16_t* p_relu = want_relu ? relu_vals + trow * (2 * G) + 2 * (g0 + g) : nullptr;
  uint16_t* p_dense = dense_out ? dense_out + trow * F + c0 + g * M : nullptr;
  uint16_t* p_rdense = relu_dense_out ? relu_dense_out + trow * F + c0 + g * M : nullptr;
  uint16_t* p_v24 = want24 ? vals24 + trow * (F >> 1) + (g0 + g) * 4 : nullptr;
  uint16_t* p_r24 = (want24 && relu24 && apply) ? relu24 + trow * (F >> 1) + (g0 + g) * 4 : nullptr;
  uint16_t* p_meta = meta + trow * (G >> 2) + ((g0 + g) >> 2);
  uint16_t* p_m24 = want24 ? meta24 + trow * (F >> 4) + ((g0 + g) >> 1) : nullptr;
  // tensor-core-ordered copies: rows of one strip share their 128-row block, so the atom is fixed
  const int64_t kw = (g0 + g) >> 2, kw24 = (g0 + g) >> 1;
  uint8_t* hw_atom = meta_hw ? meta_hw + meta_hw_offset(t0 & ~int64_t(127), kw, 4 * G) : nullptr;
  uint8_t* hw24_atom = want24 ? meta24_hw + meta_hw_offset(t0 & ~int64_t(127), kw24, F) : nullptr;
  const int s_vals = rstep * (int)(2 * G), s_dense = rstep * (int)F, s_v24 = rstep * (int)(F >> 1);
  const int s_meta = rstep * (int)(G >> 2), s_m24 = rstep * (int)(F >> 4);
  for (int r = r0; r < V; r += rstep) {
    const uint4 q = *reinterpret_cast<const uint4*>(tp);
    uint32_t rw[4] = {q.x, q.y, q.z, q.w}, hw[4];
    if (apply) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { rw[j] = relu2(rw[j]); hw[j] = sq2(rw[j]); }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) hw[j] = rw[j];
    }
    // kept columns c0 < c1 | c2 < c3 as two packed pairs
    const uint32_t a0 = __byte_perm(hw[0], hw[1], selp[0]), b0 = __byte_perm(hw[2], hw[3], selp[0]);
    const uint32_t a1 = __byte_perm(hw[0], hw[1], selp[1]), b1 = __byte_perm(hw[2], hw[3], selp[1]);
    const uint32_t hk0 = (a0 & ~mhi[0]) | (b0 & mhi[0]), hk1 = (a1 & ~mhi[1]) | (b1 & mhi[1]);
    uint32_t packed;
    const uint32_t nib = top2of4_packed(hk0, hk1, &packed);
    *reinterpret_cast<uint32_t*>(p_vals) = packed;
    // this row's pair -> its tabulated selectors (nib % 7 without a division: nib < 16)
    const uint32_t slot = nib - 7u * ((nib * 37u) >> 8);
    const uint4 sel = my_sel[slot];
    if (need_relu_pair) {
      // the two kept ReLU values straight from the group's words
      const uint32_t x = __byte_perm(rw[0], rw[1], sel.z), y = __byte_perm(rw[2], rw[3], sel.z);
      const uint32_t rpair = __byte_perm(x, y, sel.z >> 16);
      if (want_relu) *reinterpret_cast<uint32_t*>(p_relu) = rpair;
      if (p_r24) {
        // ReLU(y1) in the layout of the 2:4 view (what the dy1 epilogue multiplies by)
        *reinterpret_cast<uint2*>(p_r24) = make_uint2(__byte_perm(rpair, 0u, sel.w), __byte_perm(rpair, 0u, sel.w >> 16));
        p_r24 += s_v24;
      }
      if (relu_dense_out)
        *reinterpret_cast<uint4*>(p_rdense) = make_uint4(__byte_perm(rpair, 0u, sel.x), __byte_perm(rpair, 0u, sel.x >> 16),
                                                         __byte_perm(rpair, 0u, sel.y), __byte_perm(rpair, 0u, sel.y >> 16));
    }
    if (dense_out)
      *reinterpret_cast<uint4*>(p_dense) = make_uint4(__byte_perm(packed, 0u, sel.x), __byte_perm(packed, 0u, sel.x >> 16),
                                                      __byte_perm(packed, 0u, sel.y), __byte_perm(packed, 0u, sel.y >> 16));
    uint32_t word = nib;
    word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 4;
    word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 8;
    // offset of row r's word inside a metadata atom (r < 128)
    const uint32_t hw_row = (uint32_t)(((t0 + r) & 127) >> 4) * 256u + (uint32_t)((t0 + r) & 7) * 16u +
                            (uint32_t)(((t0 + r) >> 3) & 1) * 2u;
    if (lead4) {
      *p_meta = (uint16_t)word;
      if (hw_atom) *reinterpret_cast<uint16_t*>(hw_atom + hw_row) = (uint16_t)word;
    }
    // The same row as a plain 2:4 operand over all F columns: two values per eight columns always
    // satisfy "at most two per four", so each half-group stores its kept values (or zeros) and a
    // legal position pair. A half-group with one kept value at position p pairs it with a zero
    // at position 1 (p = 0) or 0 (p > 0).
    if (want24) {
      *reinterpret_cast<uint2*>(p_v24) = make_uint2(__byte_perm(packed, 0u, sel.w), __byte_perm(packed, 0u, sel.w >> 16));
      uint32_t mb = my_nib[slot];
      mb |= __shfl_down_sync(0xFFFFFFFFu, mb, 1) << 8;
      if (lead2) {
        *p_m24 = (uint16_t)mb;
        *reinterpret_cast<uint16_t*>(hw24_atom + hw_row) = (uint16_t)mb;
      }
      p_v24 += s_v24;
      p_m24 += s_m24;
    }
    tp += rstep * kRow;
    p_vals += s_vals;
    if (want_relu) p_relu += s_vals;
    if (dense_out) p_dense += s_dense;
    if (relu_dense_out) p_rdense += s_dense;
    p_meta += s_meta;
  }
}

}  // namespace

int launch_vnm(const void* P, int64_t T, int64_t F, int64_t ld, int V, int M, int apply_sqrelu,
               void* vals, void* meta, void* meta_hw, void* colidx, void* relu_vals, void* dense_out,
               void* relu_dense_out, void* vals24, void* meta24, void* meta24_hw, void* relu24, cudaStream_t s) {
  if (T == 0 || F == 0) return SF_OK;
  const size_t smem = (size_t)V * (kCW + kPad) * 2 + kCW * 4 + kCW + kCW;
  static bool attr_set[64] = {false};                         // per device
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(vnm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     128 * (kCW + kPad) * 2 + kCW * 6));
    SF_CUDA_TRY(cudaFuncSetAttribute(vnm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     128 * (128 + kPad) * 2 + 128 * 6));
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  dim3 grid((unsigned)((F + kCW - 1) / kCW), (unsigned)(T / V));
  // fast path: groups of eight, strips whose group count divides the thread count, full warps per row step
  const int tail = (int)(F % kCW);
  const bool fast8 = (M == 8) && (tail == 0 || tail == 64 || tail == 128) && (V % 32 == 0);
  if (fast8) {
    // 256-column strips measured as fast as 128-column ones at V = 128 and 15 % faster at V = 64
    // (the kernel is bound by instruction issue, not by resident CTAs)
    constexpr int kW8 = 256;
    static bool attr8[64] = {false};
    if (dev < 0 || dev >= 64 || !attr8[dev]) {
      SF_CUDA_TRY(cudaFuncSetAttribute(vnm8_kernel<kW8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       128 * (kW8 + kPad) * 2 + kW8 * 6 + (kW8 / 8) * 7 * 17));
      if (dev >= 0 && dev < 64) attr8[dev] = true;
    }
    const size_t smem8 = (size_t)V * (kW8 + kPad) * 2 + kW8 * 6 + (kW8 / 8) * 7 * 17;
    dim3 grid8((unsigned)((F + kW8 - 1) / kW8), (unsigned)(T / V));
    vnm8_kernel<kW8><<<grid8, kThreads, smem8, s>>>((const uint16_t*)P, T, F, ld, V, apply_sqrelu, (uint16_t*)vals,
                                                    (uint16_t*)meta, (uint8_t*)meta_hw, (uint8_t*)colidx,
                                                    (uint16_t*)relu_vals, (uint16_t*)dense_out,
                                                    (uint16_t*)relu_dense_out, (uint16_t*)vals24, (uint16_t*)meta24,
                                                    (uint8_t*)meta24_hw, (uint16_t*)relu24);
    SF_LAUNCH_CHECK();
    return SF_OK;
  }
  if (vals24) return SF_ERR_UNSUPPORTED;                 // the plain-2:4 view is produced by the fast path only
  if (M <= 32) {
    // narrow strips: 128 / M >= 4 groups per strip
    const size_t smem_n = (size_t)V * (128 + kPad) * 2 + 128 * 6;
    dim3 grid_n((unsigned)((F + 127) / 128), (unsigned)(T / V));
    vnm_kernel<128><<<grid_n, kThreads, smem_n, s>>>((const uint16_t*)P, T, F, ld, V, M, apply_sqrelu, (uint16_t*)vals,
                                                      (uint16_t*)meta, (uint8_t*)meta_hw, (uint8_t*)colidx,
                                                      (uint16_t*)relu_vals, (uint16_t*)dense_out,
                                                      (uint16_t*)relu_dense_out);
  } else {
    vnm_kernel<256><<<grid, kThreads, smem, s>>>((const uint16_t*)P, T, F, ld, V, M, apply_sqrelu, (uint16_t*)vals,
                                                  (uint16_t*)meta, (uint8_t*)meta_hw, (uint8_t*)colidx,
                                                  (uint16_t*)relu_vals, (uint16_t*)dense_out,
                                                  (uint16_t*)relu_dense_out);
  }
  SF_LAUNCH_CHECK();
  return SF_OK;
}

// True when launch_vnm can also emit the plain-2:4 view (vals24 / meta24) for this shape.
bool vnm_has_24_view(int64_t F, int V, int M) {
  const int tail = (int)(F % kCW);
  return (M == 8) && (tail == 0 || tail == 64 || tail == 128) && (V % 32 == 0);
}

}  // namespace sf
