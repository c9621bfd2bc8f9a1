// Shared host/device helpers of libsparseffn (private to csrc/).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/sparseffn.h"

namespace sf {

// Most recent failing cudaError_t (process-wide, informational).
extern int g_last_cuda_error;

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return SF_ERR_CUDA;
}

#define SF_CUDA_TRY(expr)                               \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) return ::sf::cuda_fail(_e);  \
  } while (0)

#define SF_LAUNCH_CHECK()                               \
  do {                                                  \
    cudaError_t _e = cudaGetLastError();                \
    if (_e != cudaSuccess) return ::sf::cuda_fail(_e);  \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Returns SF_OK when the current device is compute capability 10.x.
int check_arch();

// ---- bf16 bit helpers (device) ---------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// round-to-nearest-even float -> bf16 bits (finite inputs; NaN stays NaN)
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
  return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(f)));
}

// Top-2-of-4 by key (larger first, ties to the lower index). Returns the nibble
// pos0 | pos1 << 2 with pos0 < pos1; *third receives the index of the element ranked third.
__device__ __forceinline__ uint32_t top2of4(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3,
                                            uint32_t* third = nullptr) {
  // c_ij (i < j) is 1 when element i precedes element j in (key desc, index asc)
  const uint32_t c01 = k0 >= k1, c02 = k0 >= k2, c03 = k0 >= k3;
  const uint32_t c12 = k1 >= k2, c13 = k1 >= k3, c23 = k2 >= k3;
  const uint32_t r0 = (1 - c01) + (1 - c02) + (1 - c03);
  const uint32_t r1 = c01 + (1 - c12) + (1 - c13);
  const uint32_t r2 = c02 + c12 + (1 - c23);
  const uint32_t r3 = c03 + c13 + c23;
  const uint32_t keep = (r0 < 2 ? 1u : 0u) | (r1 < 2 ? 2u : 0u) | (r2 < 2 ? 4u : 0u) | (r3 < 2 ? 8u : 0u);
  const uint32_t pos0 = __ffs(keep) - 1;
  const uint32_t pos1 = 31 - __clz(keep);
  if (third) *third = (r0 == 2) ? 0u : (r1 == 2) ? 1u : (r2 == 2) ? 2u : 3u;
  return pos0 | (pos1 << 2);
}

// Same selection on a packed group (lo = elements 0,1; hi = elements 2,3; bf16 patterns), built for
// few instructions: each 15-bit magnitude is widened to magnitude*4 + (3 - index), which makes all
// four keys distinct and orders ties towards the lower index; a five-comparator network then
// yields the first, second and third key, whose low two bits name their positions.
// Returns the nibble; *packed = kept values (pos0 low half, pos1 high half); *third_idx = index of
// the third-ranked element.
__device__ __forceinline__ uint32_t top2of4_packed(uint32_t lo, uint32_t hi, uint32_t* packed,
                                                   uint32_t* third_idx = nullptr, uint32_t* perm_sel = nullptr) {
  // The integer-logic pipe is what these kernels run out of, so the widening is written as multiply-adds
  // (x * 4 + index term; x >> 14 as the high half of x * 2^18), which issue on the FMA pipe.
  const uint32_t c0 = (lo & 0x7FFFu) * 4u + 3u, c1 = __umulhi(lo & 0x7FFF0000u, 1u << 18) + 2u;
  const uint32_t c2 = (hi & 0x7FFFu) * 4u + 1u, c3 = __umulhi(hi & 0x7FFF0000u, 1u << 18);
  const uint32_t h01 = max(c0, c1), l01 = min(c0, c1), h23 = max(c2, c3), l23 = min(c2, c3);
  const uint32_t top1 = max(h01, h23), mid = min(h01, h23);
  // second overall = the larger of the losing pair-winner and the two pair-losers
  const uint32_t top2 = max(mid, max(l01, l23));
  const uint32_t ia = ~top1 & 3u, ib = ~top2 & 3u;           // 3 - (key & 3)
  const uint32_t p0 = min(ia, ib), p1 = max(ia, ib);
  // byte permute: bytes (2p0, 2p0+1) then (2p1, 2p1+1) out of the 8 bytes {lo, hi}
  const uint32_t sel = 0x1010u + p0 * 0x22u + p1 * 0x2200u;
  *packed = __byte_perm(lo, hi, sel);
  if (perm_sel) *perm_sel = sel;             // the same selector picks the pair out of any other {lo, hi}
  if (third_idx) {
    // third overall = the smaller of the losing pair-winner and the winner's partner, or the other pair's loser
    const bool first_pair_wins = h01 > h23;
    const uint32_t under = first_pair_wins ? l01 : l23, other_low = first_pair_wins ? l23 : l01;
    *third_idx = ~max(min(mid, under), other_low) & 3u;
  }
  return p1 * 4u + p0;
}

// The same selection for TWO groups at once, in the 16-bit halves of 32-bit words: x_i holds element i of
// group A in its low half and of group B in its high half (bf16 patterns). With magnitudes below 0x8000,
// (a | 0x8000) - b has bit 15 set exactly when a >= b and never borrows from the other half, so one
// subtraction compares both groups; "element i is kept" (fewer than two elements precede it in the order
// magnitude descending, index ascending) is a majority of three such flags, one logic operation each.
// The four keep flags of a group index a 16-entry table (top2_lut_init). Entry .x: low half = the
// byte-permute selector that gathers the kept pair out of {lo, hi}, high half = the metadata nibble
// replicated into all four nibbles; .y = the selector of the two dropped elements.
// Returns the entries of group A and group B.
struct Top2Entry { uint32_t kept, dropped; };
__device__ __forceinline__ Top2Entry top2_lut_entry(uint32_t keep_mask) {
  const uint32_t p0 = __ffs(keep_mask) - 1u, p1 = 31u - __clz(keep_mask);
  const uint32_t drop = ~keep_mask & 0xFu;
  const uint32_t q0 = __ffs(drop) - 1u, q1 = 31u - __clz(drop);
  return Top2Entry{(0x1010u + p0 * 0x22u + p1 * 0x2200u) | ((p0 | (p1 << 2)) * 0x11110000u),
                   0x1010u + q0 * 0x22u + q1 * 0x2200u};
}
// lut: 16 entries of shared memory; call from at least 16 threads, then synchronise.
__device__ __forceinline__ void top2_lut_init(Top2Entry* lut, int tid) {
  if (tid < 16) lut[tid] = (__popc(tid) == 2) ? top2_lut_entry((uint32_t)tid) : Top2Entry{0u, 0u};
}
// kDropped: the entries' .dropped selectors are loaded too (soft-thresholding needs the dropped pair).
template <bool kDropped = false>
__device__ __forceinline__ void top2of4_x2(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3, const Top2Entry* lut,
                                           Top2Entry& entry_a, Top2Entry& entry_b) {
  constexpr uint32_t kMag = 0x7FFF7FFFu, kTop = 0x80008000u;
  const uint32_t m1 = x1 & kMag, m2 = x2 & kMag, m3 = x3 & kMag;
  const uint32_t o0 = x0 | kTop, o1 = x1 | kTop, o2 = x2 | kTop;
  const uint32_t g01 = o0 - m1, g02 = o0 - m2, g03 = o0 - m3, g12 = o1 - m2, g13 = o1 - m3, g23 = o2 - m3;
  // element j < i precedes i when m_j >= m_i; element j > i precedes i when not (m_i >= m_j)
  const uint32_t k0 = (g01 & g02) | (g01 & g03) | (g02 & g03);
  const uint32_t k1 = (~g01 & g12) | (~g01 & g13) | (g12 & g13);
  const uint32_t k2 = (~g02 & ~g12) | (~g02 & g23) | (~g12 & g23);
  const uint32_t k3 = ~((g03 & g13) | (g03 & g23) | (g13 & g23));
  // flags (bits 15 and 31) -> byte offsets into the table (bits 3..6 of either half)
  const uint32_t t = ((k0 >> 12) & 0x00080008u) | ((k1 >> 11) & 0x00100010u) | ((k2 >> 10) & 0x00200020u) |
                     ((k3 >> 9) & 0x00400040u);
  const uint8_t* base = reinterpret_cast<const uint8_t*>(lut);
  if (kDropped) {
    const uint2 a = *reinterpret_cast<const uint2*>(base + (t & 0xFFFFu)), b = *reinterpret_cast<const uint2*>(base + (t >> 16));
    entry_a = Top2Entry{a.x, a.y};
    entry_b = Top2Entry{b.x, b.y};
  } else {
    entry_a = Top2Entry{*reinterpret_cast<const uint32_t*>(base + (t & 0xFFFFu)), 0u};
    entry_b = Top2Entry{*reinterpret_cast<const uint32_t*>(base + (t >> 16)), 0u};
  }
}
// Soft-thresholding (Section 2.2) of a group's kept pair, given the group as {lo, hi} and its table entry:
// the threshold is the larger magnitude of the two dropped elements; every kept value moves towards zero
// by it (never across: kept magnitudes are at least the threshold). The packed bf16 subtraction rounds
// the exact difference once, which equals the float32 subtraction followed by rounding to bf16 (the
// float32 result is exact unless the threshold is below 2^-16 of the value, where both give the value
// itself). A kept NaN is neither above nor below the threshold and becomes zero.
__device__ __forceinline__ uint32_t soft_threshold_pair(uint32_t lo, uint32_t hi, const Top2Entry& e) {
  const uint32_t kept = __byte_perm(lo, hi, e.kept);
  const uint32_t dm = __byte_perm(lo, hi, e.dropped) & 0x7FFF7FFFu;
  const uint32_t t = max(dm & 0xFFFFu, dm >> 16);
  const uint32_t ct = (kept & 0x80008000u) | (t * 0x00010001u);          // the threshold with each value's sign
  const __nv_bfloat162 d = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&kept), *reinterpret_cast<const __nv_bfloat162*>(&ct));
  const __nv_bfloat162 kv = *reinterpret_cast<const __nv_bfloat162*>(&kept);
  return *reinterpret_cast<const uint32_t*>(&d) & ~__hneu2_mask(kv, kv);
}

// ---- internal launchers (defined in the .cu files) ---------------------------------------
// meta_hw (optional) receives the same metadata words in the order the sparse tensor-core
// instruction reads them (see meta_hw_offset below); requires R % 128 == 0 and K % 128 == 0.
int launch_prune24(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim, int prune_mode,
                   void* vals, void* meta, void* meta_hw, void* dense_out, cudaStream_t s);
int launch_vnm(const void* P, int64_t T, int64_t F, int64_t ld, int V, int M, int apply_sqrelu,
               void* vals, void* meta, void* meta_hw, void* colidx, void* relu_vals, void* dense_out,
               void* relu_dense_out, void* vals24, void* meta24, void* meta24_hw, void* relu24, cudaStream_t s);
// Strided groups with the kept values quantised to E4M3 codes in the same pass (vals uint8 [cols, rows/2]).
int launch_prune24_cols_fp8(const void* W, int64_t rows, int64_t cols, int64_t ld, int prune_mode, float scale, void* vals,
                            void* meta, cudaStream_t s);
bool vnm_has_24_view(int64_t F, int V, int M);
// Streaming form of the sparsifier (values, ReLU values, canonical metadata and colidx only).
bool vnm_stream_supported(int64_t F, int64_t ld, int V, int M, const void* P);
int launch_vnm_stream(const void* P, int64_t T, int64_t F, int64_t ld, int V, int M, int apply_sqrelu, void* vals,
                      void* meta, void* colidx, void* relu_vals, cudaStream_t s);
int launch_transpose(const void* in, void* out, int64_t rows, int64_t cols, cudaStream_t s);
// Device address of the status word of the built-in scratch array (sf_gemm_sparse24_noalloc).
int noalloc_status_word(void** out);
// Records the next caller-owned trace event on `s` while stage tracing is on (sf_trace_set); else a no-op.
void trace_mark(cudaStream_t s);

// Byte offset of the metadata word (row m, 16-column word kw) inside the hardware-ordered
// metadata tensor of a [R, K] 2:4 operand: 2 KB atoms of 128 rows x 128 columns, atoms of one
// row block stored consecutively along K.
__host__ __device__ __forceinline__ size_t meta_hw_offset(int64_t m, int64_t kw, int64_t K) {
  const int64_t atoms_per_rowblock = K >> 7;
  const int64_t atom = (m >> 7) * atoms_per_rowblock + (kw >> 3);
  const int mi = static_cast<int>(m & 127), kwi = static_cast<int>(kw & 7);
  return static_cast<size_t>(atom) * 2048 + (mi >> 4) * 256 + (kwi & 1) * 128 + (mi & 7) * 16 +
         (kwi >> 1) * 4 + ((mi >> 3) & 1) * 2;
}

// The same for an 8-bit (E4M3) 2:4 operand: per 128 rows and 256 columns a pair of 2 KB atoms (128 columns
// each); inside an atom the rows are plain: 16 bytes per row, the eight 16-column words in order.
__host__ __device__ __forceinline__ size_t meta_hw8_offset(int64_t m, int64_t kw, int64_t K) {
  const int64_t pairs_per_rowblock = K >> 8;
  const int64_t pair = (m >> 7) * pairs_per_rowblock + (kw >> 4);
  const int mi = static_cast<int>(m & 127), kwi = static_cast<int>(kw & 15);
  return static_cast<size_t>(pair) * 4096 + (kwi >> 3) * 2048 + mi * 16 + (kwi & 7) * 2;
}

}  // namespace sf
