// Internal interface of the tensor-core products (gemm_tc.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sf {

enum GemmMode { MODE_DENSE = 0, MODE_SPARSE24 = 1, MODE_VENOM = 2 };

enum GemmEpilogue {
  EPI_STORE = 0,    // C[m, n] = bf16(acc)
  EPI_SQRELU = 1,   // C = y = bf16(acc);  C2 = bf16(max(y, 0)^2)                     (Eq. 2)
  EPI_DRELU = 2,    // C = bf16(2 * acc * max(aux[m, n], 0))                           (Eq. 6)
  EPI_STORE_T = 3,  // C[n, m] = bf16(acc)          (accumulator rows are output columns)
  EPI_DRELU_T = 4,  // C[n, m] = bf16(2 * acc * aux[n, m]), +0 where aux is zero       (Eq. 6 on the mask)
  EPI_VNM8 = 5,     // SquaredReLU + V:N:M selection (groups of eight) on the accumulator tile itself: rows are
                    // features, columns are tokens; writes the packed activation, never the dense y1  (Eq. 2, Section 2.3)
  EPI_DRELU24_T = 6,// as EPI_DRELU_T with aux given in the 2:4 layout of the mask (values [n, m/2] + pack_meta) and
                    // only the packed output written
  EPI_ACT24_T = 7,  // transposed output with SquaredReLU and a 2:4 selection inside every four features of a token
                    // (the routed step's activation, Section 3.1 step 3): packed values, packed ReLU values, both
                    // metadata orders and the masked dense copy; never the pre-activation unless asked for
  EPI_ROUTE = 8     // accumulator rows are tokens, its first route_E columns the experts' logits: each row writes its
                    // arg-max (ties to the lower expert) and, optionally, the float32 logits   (Section 3.1 step 1)
};

// One output tile of a table-driven (grouped) product on CTA pairs. Offsets are in elements of the
// operand's own coordinates: a_row / b_row select the 256 (A) or tile-width (B) rows or columns the tile
// reads, a_k0 / b_k0 where its reduction range starts in either operand, nkb how many k-blocks (of 128
// logical K for 2:4 products, 64 for dense ones) it spans; out_m / out_n are the output coordinates the
// epilogue uses (they differ from a_row / b_row when an operand is a slice of a larger matrix), n_limit
// the first output column that does not belong to the tile's group any more.
struct GemmTile {
  int a_row, a_k0, b_row, b_k0, nkb, out_m, out_n, n_limit;
};

struct GemmArgs {
  int64_t M, N, K;
  void* C;
  int64_t ldc;
  void* C2;
  int64_t ldc2;
  const void* aux;
  int64_t ldaux;
  const uint8_t* meta_hw;   // sparse modes: hardware-ordered metadata atoms
  const uint8_t* colidx;    // Venom: [T/V, G, 4]
  int64_t G;                // Venom: groups per row (F / Mv)
  int V, Mv;                // Venom block height and group width
  int* status;              // device status word (set to 1 when a bounded wait expires)
  int num_m_tiles, num_n_tiles, num_k_blocks;
  int gather_tma_groups;    // Venom: groups (of 16 per stage) fetched by TMA row gather; the rest by cp.async
  // EPI_DRELU_T only, optional: also emit the output packed as a 2:4 operand at given positions
  const void* pack_meta;    // canonical 2:4 metadata [N, M/16] uint16 (rows = output rows of Ct)
  void* pack_vals;          // bf16 [N, M/2]
  // EPI_VNM8 outputs (T = N tokens, F = M features, G = F / 8 groups per token)
  void* vn_vals;            // bf16 [T, 2G]   kept activation values (V:N:M packed)
  void* vn_relu;            // bf16 [T, 2G]   ReLU(y1) at the same positions
  void* vn_meta;            // uint16 [T, G/4] canonical nibbles over the condensed matrix
  void* vn_colidx;          // uint8 [T/V, G, 4]
  void* vn_vals24;          // bf16 [T, F/2]  the same activation as a plain 2:4 operand over all F columns
  void* vn_relu24;          // bf16 [T, F/2]  ReLU(y1) in that layout
  void* vn_meta24;          // uint16 [T, F/16] canonical metadata of that operand
  void* vn_meta24_hw;       // the same words in tensor-core order
  void* vn_y1;              // optional bf16 [T, F]: the pre-activation itself
  void* vn_dense;           // optional bf16 [T, F]: the activation on its mask, +0 elsewhere
  // table-driven tiles (grouped products of the routed step); null = the regular tile raster
  const GemmTile* tile_table;
  const int* num_tiles_dev;  // device word holding the number of valid entries of tile_table
  // EPI_STORE only, optional: output row r of the product is written to row row_map[r] of C (skipped when < 0)
  const int* row_map;
  // EPI_STORE only: the accumulator is multiplied by this before rounding (0 = no scaling)
  float out_scale;
  // EPI_ROUTE
  int* route_expert;         // int32 [M]
  float* route_logits;       // optional float32 [M, route_E]
  int route_E;               // 1..16
};

// Outputs of the fused y1 product (see GemmArgs::vn_*).
struct Vnm8Out {
  void *vals, *relu, *meta, *colidx, *vals24, *relu24, *meta24, *meta24_hw, *y1, *dense;
};

// D[M,N] = op(A) op(B)^T, tiles 128 x 256, K % 64 == 0.
int gemm_dense(const void* A, bool a_kmajor, const void* B, bool b_kmajor, int64_t M, int64_t N, int64_t K, int epi,
               void* C, int64_t ldc, void* C2, int64_t ldc2, const void* aux, int64_t ldaux, int* status,
               cudaStream_t s);
// The weight-gradient products with one operand given packed: D[M,N] = A^T B with A [K, M] and B [K, N]
// row-major (reduction over the rows), where operand `packed_operand` (1 = A, 2 = B) is not read as a
// dense matrix but expanded on the fly from its 2:4 layout: values [K, X/2] + canonical metadata
// [K, X/16] (X = M or N). M % 256 == 0, N % 256 == 0, K % 64 == 0.
int gemm_dense_expand(const void* dense_op, int packed_operand, const void* pk_vals, const void* pk_meta, int64_t M,
                      int64_t N, int64_t K, void* C, int64_t ldc, int* status, cudaStream_t s);
// y1 product with the activation sparsified in the epilogue: W1s [F, D] 2:4-packed times X [T, D];
// F % 256 == 0, D % 128 == 0, T % V == 0, V in {64, 128}. Nothing of y1 is written unless out.y1 is set.
int gemm_sparse24_vnm8(const void* a_vals, const uint8_t* meta_hw, const void* X, int64_t F, int64_t T, int64_t D,
                       int V, const Vnm8Out& out, int* status, cudaStream_t s);
bool gemm_sparse24_vnm8_supported(int64_t F, int64_t T, int64_t D, int V);

// ---- grouped products of the routed step (tile tables built on the device, see router.cu) ------------------
// Outputs of the routed y1 product's epilogue, all indexed [row of the permuted token order, local feature]
// with Fe = features per expert: values / ReLU values [rows, Fe/2], canonical metadata [rows, Fe/16] and its
// tensor-core order, masked dense copy [rows, Fe], optional pre-activation [rows, Fe].
struct Act24Out {
  void *vals, *relu, *meta, *meta_hw, *dense, *y1;
};
// y1c = Xp W1s[expert block]^T with the epilogue above. a_vals/meta_hw: W1s [F, D] packed; Xp [rows, D].
int gemm_grouped_act24(const void* a_vals, const uint8_t* meta_hw, const void* Xp, int64_t rows, int64_t F, int64_t Fe,
                       int64_t D, const Act24Out& out, const GemmTile* tiles, const int* num_tiles, int max_tiles,
                       int* status, cudaStream_t s);
// dy1c = 2 (dYp W2s[expert block]) ReLU(y1c) on the mask: packed (pack_vals) and masked dense (C) copies.
int gemm_grouped_drelu24(const void* a_vals, const uint8_t* meta_hw, const void* dYp, int64_t rows, int64_t F,
                         int64_t Fe, int64_t D, const void* relu_vals, const void* meta, void* pack_vals, void* dense,
                         const GemmTile* tiles, const int* num_tiles, int max_tiles, int* status, cudaStream_t s);
// C[rows, N] = A_s[rows, Fe] (2:4-packed activations) times the expert's slice of a weight matrix:
// b_kmajor: B = W [N, Ktot] row-major (slice of columns); else B = W [Ktot, N] row-major (slice of rows).
// row_map (optional): row r of the product lands in row row_map[r] of C, rows mapped to -1 are dropped (the
// un-grouping of the routed step's outputs, done by the epilogue's own stores).
int gemm_grouped_sparse24_rm(const void* a_vals, const uint8_t* meta_hw, const void* B, bool b_kmajor, int64_t rows,
                             int64_t N, int64_t Fe, int64_t Ktot, void* C, const int* row_map, const GemmTile* tiles,
                             const int* num_tiles, int max_tiles, int* status, cudaStream_t s);
// C[M, N] (leading dimension ldc) accumulates A^T B over each tile's own range of rows: A [rows, Ma], B [rows, Nb]
// row-major (both reduced over rows).
int gemm_grouped_dense_tn(const void* A, int64_t Ma, const void* B, int64_t Nb, int64_t rows, void* C, int64_t ldc,
                          const GemmTile* tiles, const int* num_tiles, int max_tiles, int* status, cudaStream_t s);
// A_s[M,K] 2:4-packed times B (b_kmajor: [N,K] row-major, else [K,N] row-major).
// epi EPI_STORE_T / EPI_DRELU_T: transposed output Ct[N,M] (b_kmajor only); EPI_STORE: C[M,N]
// (two-CTA kernel, M % 256 == 0).
// pack_meta / pack_vals (EPI_DRELU_T, optional): additionally write Ct gathered at the positions of the
// canonical 2:4 metadata pack_meta [N, M/16] into pack_vals [N, M/2].
int gemm_sparse24(const void* a_vals, const uint8_t* meta_hw, const void* B, bool b_kmajor, int64_t M, int64_t N,
                  int64_t K, int epi, void* C, int64_t ldc, const void* aux, int64_t ldaux, int* status,
                  cudaStream_t s, const void* pack_meta = nullptr, void* pack_vals = nullptr);
// Routing on the tensor cores: logits[T, E] = X[T, D] means[E, D]^T in float32 accumulators, the arg-max per token
// taken in the epilogue (ties to the lower expert). T % 256 == 0, D % 64 == 0, 1 <= E <= 16; the means need no
// padding (rows beyond E are read as zeros by the tensor map).
int gemm_route(const void* X, const void* means, int64_t T, int64_t D, int E, int* expert, float* logits, int* status,
               cudaStream_t s);
// E4M3 operands, both K-major: C[M, N] = bf16(alpha * A B^T). sparse: A = 2:4 values [M, K/2] (codes) with
// metadata in the 8-bit instruction's order (see meta_hw8_offset); else A [M, K]. B [N, K].
// M % 256 == 0, N % 32 == 0, K % 256 == 0 (2:4) or K % 128 == 0 (dense).
int gemm_fp8(bool sparse, const void* A, const uint8_t* meta_hw, const void* B, int64_t M, int64_t N, int64_t K,
             float alpha, void* C, int64_t ldc, int* status, cudaStream_t s);
// C[T,N] = A_vnm[T,F] Bt[F,N]; A_vnm packed (vals [T, 2F/Mv], hardware-ordered metadata, colidx).
int gemm_venom(const void* a_vals, const uint8_t* meta_hw, const uint8_t* colidx, const void* Bt, int64_t T,
               int64_t F, int64_t N, int V, int Mv, void* C, int64_t ldc, int* status, cudaStream_t s);

// 2D TMA descriptor (a CUtensorMap, 128 bytes, 64-byte aligned) over a row-major [rows, cols] matrix of 2-byte
// elements with leading dimension ld; box = {box_cols, box_rows}.
int make_tmap_2d(void* map, const void* base, int64_t rows, int64_t cols, int64_t ld, uint32_t box_cols,
                 uint32_t box_rows, bool swizzle128);

// canonical [R, K/16] metadata words -> hardware-ordered atoms (R % 128 == 0, K % 128 == 0)
int launch_meta_reorder(const void* meta, void* meta_hw, int64_t R, int64_t K, cudaStream_t s);
// dy1 packing: gather a dense [T, F] matrix at the positions recorded by (colidx, meta)
int launch_pack_like(const void* dense, const void* meta, const void* colidx, void* vals, int64_t T, int64_t F,
                     int V, int Mv, cudaStream_t s);

}  // namespace sf
