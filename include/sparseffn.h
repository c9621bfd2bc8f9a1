/*
 * sparseffn.h — C ABI of libsparseffn.so: the sparsified Transformer-FFN training step on
 * NVIDIA B200 (sm_100a).
 *
 * The step (paper: Algorithms 1 and 2, Sections 2.1-2.3, 3) re-prunes the FFN weights to 2:4
 * every iteration, computes SquaredReLU(X W1^T), sparsifies the activation into the V:N:M
 * (Venom) format and runs the forward/backward products with exactly one sparse operand each.
 *
 * Conventions for every entry point
 *   - Tensors are row-major bf16 (16-bit patterns) unless stated. T = tokens, D = d_model,
 *     F = d_ffn.  X [T,D], W1 [F,D], W2 [D,F], Y/dY [T,D]  (the paper writes the weights
 *     transposed, W1 [D,F], W2 [F,D]; the mathematics is the same).
 *   - Pointers are DEVICE pointers owned by the caller unless the name says "host". The
 *     library never allocates or frees device memory and never synchronises, except where an
 *     entry point says so. Work is enqueued on the caller's stream (`stream` is a
 *     cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - Return value: SF_OK (0) or a negative sf_status. No exceptions cross the boundary. Argument
 *     errors (NULL, shape, alignment, workspace size, architecture) are found before anything is
 *     enqueued; after an SF_ERR_CUDA some kernels of the call may already be enqueued and the
 *     outputs are undefined.
 *   - Base pointers must be 16-byte aligned and leading dimensions multiples of 8 elements.
 *   - Canonical 2:4 metadata: one nibble per group of four, `pos0 | pos1 << 2` with
 *     pos0 < pos1 the kept positions; four consecutive groups of a row are packed
 *     little-endian into one uint16.
 */
#ifndef SPARSEFFN_H_
#define SPARSEFFN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SF_API __attribute__((visibility("default")))
#else
#define SF_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum sf_status {
  SF_OK = 0,
  SF_ERR_NULL = -1,      /* a required pointer is NULL */
  SF_ERR_SHAPE = -2,     /* a size violates the divisibility rules stated per call */
  SF_ERR_ALIGN = -3,     /* base pointer not 16-byte aligned or ld not a multiple of 8 */
  SF_ERR_WORKSPACE = -4, /* workspace / context too small */
  SF_ERR_ARCH = -5,      /* current device is not compute capability 10.x */
  SF_ERR_CUDA = -6,      /* a CUDA call failed; see sf_last_cuda_error() */
  SF_ERR_TIMEOUT = -7,   /* a bounded device-side wait expired (reported by sf_check_status) */
  SF_ERR_UNSUPPORTED = -8 /* legal per the paper but not built (e.g. N != 2) */
} sf_status;

/* Problem descriptor of one FFN layer step. Ragged shapes are rejected, never padded:
 * T, D, F multiples of 128 and at least 256 (every product runs on 256-row tiles of a CTA pair; the
 * last pair of a product may be half empty), T % V == 0, F % (4 M) == 0, V in {64,128}, N == 2,
 * M in {4,8,16,32,64}. With M >= 16 (products on the gathered Venom kernel) or with
 * SF_FFN_PACKED_GRAD_OPERANDS: multiples of 256, and (4F/M) % 128 == 0 for M >= 16. */
typedef enum sf_ffn_flags {
  SF_FFN_SAVE_Y1 = 1,     /* also store the full bf16 pre-activation y1 in the context (SF_CTX_Y1) */
  SF_FFN_UNFUSED_ACT = 2, /* M == 8: run SquaredReLU + V:N:M as its own kernel on a stored y1, never inside the
                             y1 product's epilogue */
  SF_FFN_FUSED_ACT = 4,   /* M == 8: run them inside the y1 product's epilogue whenever the shape allows. With
                             neither bit the library fuses for V == 64 (token tiles of three blocks) and not for
                             V == 128 (a one-block tile re-reads the weight operand too often). Same results
                             either way, bit for bit. */
  SF_FFN_PACKED_GRAD_OPERANDS = 8 /* M == 8: keep no masked [T, F] copy of y2 and dy1; the two weight-gradient
                             products expand their operand from its packed form inside the kernel. Saves
                             4*T*F bytes of context + workspace, costs about a third more time in those two
                             products. Same results, bit for bit. */,
  SF_FFN_W2_FD = 16 /* W2 is given, and dW2 is returned, as [F, D] row-major (the transposed storage) in every
                       step call of this descriptor, the dense step included. The 2:4 groups of W2 along d_model
                       are then contiguous (the faster pruning pass), and the M >= 16 step needs no transposed
                       copy of W2. Without the flag W2 and dW2 are [D, F]. */
} sf_ffn_flags;
typedef struct sf_ffn_desc {
  int64_t T, D, F;
  int32_t V, N, M;
  int32_t prune_mode;  /* 0: hard magnitude top-2-of-4; 1: soft-thresholding (Section 2.2) */
  int32_t flags;       /* OR of sf_ffn_flags; other bits are rejected with SF_ERR_UNSUPPORTED */
} sf_ffn_desc;

SF_API const char* sf_status_string(int status);
/* cudaError_t value of the most recent failed CUDA call made by this library (per process). */
SF_API int sf_last_cuda_error(void);

/* ---------------------------------------------------------------------------------------
 * 2:4 weight sparsification (Section 2.2; Section 3.2.1 "packed format along with sparsity
 * metadata"; Algorithm 1 line 4, Algorithm 2 line 2).
 *
 * Per group of four consecutive elements along the chosen dimension keep the two largest
 * magnitudes (ties to the lower index); prune_mode 1 additionally subtracts the group's
 * second-smallest magnitude from the kept magnitudes (soft-thresholding).
 *
 *   W          [rows, cols] bf16, leading dimension ld (elements)
 *   group_dim  1: groups along a row (contiguous);   R = rows, K = cols
 *              0: groups along a column (strided);   R = cols, K = rows; outputs are written
 *                 K-major, i.e. as for the transposed matrix
 *   vals       out, bf16 [R, K/2]   kept values in position order
 *   meta       out, uint16 [R, K/16] canonical metadata
 *   dense_out  optional out (may be NULL): the pruned matrix in the input's own layout
 *              [rows, cols] with leading dimension cols, dropped entries +0
 * Shape rules: K % 16 == 0; group_dim 0 additionally needs cols % 8 == 0.
 * sf_prune24_sizes reports the byte sizes of vals and meta.
 */
SF_API int sf_prune24_sizes(int64_t rows, int64_t cols, int group_dim, size_t* vals_bytes, size_t* meta_bytes);
SF_API int sf_prune24_compress(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim,
                        int prune_mode, void* vals, void* meta, void* dense_out, void* stream);

/* ---------------------------------------------------------------------------------------
 * SquaredReLU + V:N:M activation sparsification (Eq. 2; Section 2.3; Table 5; Algorithm 1
 * lines 5-6 with magnitude selection in place of the learned router).
 *
 * The [T,F] input is cut into blocks of V rows x M columns. Per block the four columns with
 * the largest score stay, where score = sum over the block's rows (first to last, float32) of
 * |h|, h = bf16(max(p,0)^2) when apply_sqrelu != 0, else h = p; ties to the lower column.
 * Per row the two largest magnitudes among those four columns stay (ties to the lower one).
 *
 *   preact     [T, F] bf16, leading dimension ld
 *   vals       out, bf16 [T, 2F/M]        kept h values, position order
 *   meta       out, uint16 [T, F/(4M)]    canonical nibbles over the condensed [T, 4F/M] matrix
 *   colidx     out, uint8 [T/V, F/M, 4]   kept columns per block, ascending, each < M
 *   relu_vals  optional out, bf16 [T, 2F/M]: max(p,0) at the kept positions (needed by the
 *              backward pass; ignored when apply_sqrelu == 0)
 *   dense_out  optional out, bf16 [T, F]: h on the mask, +0 elsewhere
 * Shape rules: N == 2; M in {4,8,16,32,64}; T % V == 0; V in [1,128]; F % (4*M) == 0; F % 64 == 0.
 */
SF_API int sf_vnm_sizes(int64_t T, int64_t F, int V, int N, int M,
                 size_t* vals_bytes, size_t* meta_bytes, size_t* colidx_bytes);
SF_API int sf_vnm_sparsify_act(const void* preact, int64_t T, int64_t F, int64_t ld, int V, int N, int M,
                        int apply_sqrelu, void* vals, void* meta, void* colidx, void* relu_vals,
                        void* dense_out, void* stream);

/* ---------------------------------------------------------------------------------------
 * Single products on the tensor cores (the building blocks of Algorithms 1 and 2, exposed for
 * parity tests and for the 2:4 / Venom micro-benchmarks of Section 5.2.3).
 *
 * sf_gemm_dense:  C[Mr,Nc] = op(A) op(B)^T, fp32 accumulate, bf16 out.
 *     a_kmajor = 1: A is [Mr,K] row-major;  0: A is stored [K,Mr] row-major (M contiguous)
 *     b_kmajor = 1: B is [Nc,K] row-major;  0: B is stored [K,Nc] row-major (N contiguous)
 *     Mr % 128 == 0, Nc % 256 == 0, K % 64 == 0.
 * sf_gemm_sparse24:  Ct[Nc,Mr] (transposed output!) with C[Mr,Nc] = A_s[Mr,K] B[Nc,K]^T where
 *     A_s is given packed: a_vals bf16 [Mr,K/2], a_meta canonical uint16 [Mr,K/16].
 *     This is y1 = X W1s^T with A_s = W1s, B = X, output y1 [T,F].  Mr % 128, Nc % 256, K % 128.
 * sf_gemm_sparse24_rm:  C[Mr,Nc] (row-major) = A_s[Mr,K] op(B)^T with the same packed A_s;
 *     b_kmajor = 1: B is [Nc,K] row-major; 0: B is stored [K,Nc] row-major. This is how V:N:M
 *     activations with M <= 8 are multiplied: every such row is also a legal 2:4 row over all F
 *     columns (y3 = y2 W2^T with B = W2 as stored; dX = dy1 W1 with B = W1 as stored).
 *     Mr % 256, Nc % 256, K % 128.
 * sf_gemm_venom:  C[T,Nc] = A_vnm[T,F] Bt[F,Nc] with A_vnm in V:N:M packed form (vals, meta,
 *     colidx as produced by sf_vnm_sparsify_act) and Bt row-major [F,Nc] (rows are gathered by
 *     colidx).  T % 128, V in {64,128}, Nc % 256, (4F/M) % 128 == 0.
 * `workspace` needs sf_gemm_workspace_size() bytes (hardware-ordered metadata copy + status).
 */
SF_API int sf_gemm_workspace_size(int64_t Mr, int64_t K, size_t* bytes);
SF_API int sf_gemm_dense(const void* A, int a_kmajor, const void* B, int b_kmajor, void* C,
                  int64_t Mr, int64_t Nc, int64_t K, void* workspace, void* stream);
SF_API int sf_gemm_sparse24(const void* a_vals, const void* a_meta, const void* B, void* Ct,
                     int64_t Mr, int64_t Nc, int64_t K, void* workspace, void* stream);
SF_API int sf_gemm_sparse24_rm(const void* a_vals, const void* a_meta, const void* B, int b_kmajor, void* C,
                               int64_t Mr, int64_t Nc, int64_t K, void* workspace, void* stream);
SF_API int sf_gemm_venom(const void* a_vals, const void* a_meta, const void* colidx, const void* Bt,
                  void* C, int64_t T, int64_t F, int64_t Nc, int V, int M,
                  void* workspace, void* stream);

/* sf_gemm_sparse24_noalloc: the same product as sf_gemm_sparse24 for callers that cannot allocate
 * device memory (the paper has no counterpart; this is a deployment variant). Some callers only
 * own their input and output buffers: code that runs inside another framework's allocator or
 * stream callback, plugins that are handed tensors but no allocator, processes whose device pool
 * is already fully committed. For them the scratch that sf_gemm_sparse24 takes as `workspace`
 * (metadata in tensor-core order + status word) is a 4 MiB + 256 B device array built into the
 * library; every GPU that loads the library holds it until the process exits.
 *   - Limit: Mr * K / 8 <= 4 MiB (e.g. 4096 x 8192); larger shapes return SF_ERR_WORKSPACE.
 *   - The call itself allocates and frees nothing (no cudaMalloc / cudaFree, no allocating
 *     library routine). Inputs and output are the caller's, exactly as for sf_gemm_sparse24.
 *   - The first call on each device looks up the array's device address, and that is also the
 *     moment the CUDA runtime loads the module that contains the array (4 MiB + 256 B of device
 *     memory, taken once per device by the runtime, not by this code). Make that first call at
 *     start-up, outside any stream capture, from one host thread; later calls take no memory.
 *   - All calls share the one array: two calls that may overlap on the GPU (different streams,
 *     or different host threads) race on it. Serialise them on one stream.
 *   - A bounded-wait expiry is recorded in the array's own status word, which every call clears
 *     before its kernels start; sf_check_status(NULL, stream) reads it (and allocates nothing). */
SF_API int sf_gemm_sparse24_noalloc(const void* a_vals, const void* a_meta, const void* B, void* Ct,
                                    int64_t Mr, int64_t Nc, int64_t K, void* stream);

/* ---------------------------------------------------------------------------------------
 * FP8 (E4M3) operands with the quantisation folded into the pass that already scans the matrix
 * (Section 3.2.2, last paragraph; the paper names the idea and fixes no format or scaling).
 * As built: E4M3 codes (1-4-3 bits, bias 7, no infinities, |max| = 448), one float32 scale per
 * tensor supplied by the caller; code = e4m3(float(x) * scale) with one float32 product and one
 * conversion (round to nearest even, magnitudes above 448 and infinities clamp to 448, a NaN gives
 * a NaN code). Device pointers; `ld` in elements.
 *
 * sf_fp8_quantize: Xq[r, c] = code of X[r, c]. X bf16 [rows, cols] (ld >= cols, ld % 8 == 0),
 *     Xq uint8 [rows, cols] contiguous. cols % 16 == 0.
 * sf_prune24_compress_fp8: the 2:4 pass of sf_prune24_compress (same group_dim convention, same
 *     selection, same soft-threshold shrinkage rounded to bf16) whose kept values leave as codes:
 *     vals uint8 [R, K/2], meta uint16 [R, K/16] (canonical, identical to the bf16 pass; R, K as
 *     for sf_prune24_compress). group_dim = 1: cols % 32 == 0, optional dense_out uint8
 *     [rows, cols] (codes on the mask, +0 elsewhere). group_dim = 0: rows % 16 == 0, cols % 8 == 0,
 *     dense_out must be NULL (SF_ERR_UNSUPPORTED otherwise). 2 B read + 0.625 B written per element.
 * sf_gemm_fp8_dense:    C[Mr,Nc] = bf16(alpha * A B^T), A uint8 [Mr,K], B uint8 [Nc,K] (codes).
 * sf_gemm_fp8_sparse24: the same with A given 2:4-packed: a_vals uint8 [Mr,K/2], a_meta canonical
 *     uint16 [Mr,K/16]. alpha is normally 1 / (scale_A * scale_B).
 *     Mr % 256 == 0, Nc % 256 == 0, K % 128 == 0 (dense) or K % 256 == 0 (2:4). fp32 accumulation.
 * `workspace`: sf_gemm_fp8_workspace_size(Mr, K) bytes (status word + metadata in the order the
 *     8-bit 2:4 instruction reads it); read its status with sf_check_status.
 * Errors as everywhere: SF_ERR_SHAPE / NULL / ALIGN / ARCH before anything is launched. */
SF_API int sf_fp8_quantize(const void* X, int64_t rows, int64_t cols, int64_t ld, float scale, void* Xq, void* stream);
SF_API int sf_prune24_fp8_sizes(int64_t rows, int64_t cols, int group_dim, size_t* vals_bytes, size_t* meta_bytes);
SF_API int sf_prune24_compress_fp8(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim, int prune_mode,
                                   float scale, void* vals, void* meta, void* dense_out, void* stream);
SF_API int sf_gemm_fp8_workspace_size(int64_t Mr, int64_t K, size_t* bytes);
SF_API int sf_gemm_fp8_dense(const void* A, const void* B, void* C, int64_t Mr, int64_t Nc, int64_t K, float alpha,
                             void* workspace, void* stream);
SF_API int sf_gemm_fp8_sparse24(const void* a_vals, const void* a_meta, const void* B, void* C, int64_t Mr, int64_t Nc,
                                int64_t K, float alpha, void* workspace, void* stream);

/* ---------------------------------------------------------------------------------------
 * The FFN step (Algorithm 1 = forward, Algorithm 2 = backward; Eqs. 1-8 for the dense phase).
 *
 * sf_ffn_workspace_size: bytes of the forward context (saved for backward) and of the scratch
 * workspace for `desc` (each the larger of what the sparse and the dense step need). Both buffers
 * are caller-allocated device memory, 256-byte aligned. The first 256 bytes of a workspace hold
 * the device status word: zero them once before first use. Every step call takes the sizes of the
 * two buffers it is given and returns SF_ERR_WORKSPACE, before enqueuing anything, when one is
 * smaller than the descriptor needs.
 *
 * sf_sparse_ffn_fwd:  W1s = prune24(W1 along D);  y1 = X W1s^T;  y2 = V:N:M(ReLU(y1)^2);
 *                     Y = y2 W2^T  (W2 dense).  Saves packed y2, packed ReLU(y1), metadata,
 *                     column indices (and y1 with SF_FFN_SAVE_Y1) in fwd_ctx.
 *                     M == 8: SquaredReLU and the V:N:M selection run inside the epilogue of the y1
 *                     product on the accumulator tile (y1 is never written); the activation is also
 *                     kept as a plain 2:4 operand over all F columns (two of eight is at most two
 *                     of four), which is what the products consume: identical results, no row
 *                     gather. ReLU(y1) exists in that layout only.
 *                     M >= 16: the product consumes the condensed V:N:M operand and gathers the kept
 *                     rows of W2^T.
 * sf_sparse_ffn_bwd:  W2s = prune24(W2 along D);  dy2 = dY W2s;  dy1 = 2 dy2 ReLU(y1) on y2's
 *                     mask;  dX = dy1 W1 (W1 dense);  dW1 = dy1^T X [F,D];  dW2 = dY^T y2 [D,F].
 *                     The two weight-gradient products reduce over tokens, so they run on the dense
 *                     tensor path on a masked [T, F] copy of y2 / dy1 written by the epilogue that
 *                     produces it (or, with SF_FFN_PACKED_GRAD_OPERANDS, on the packed form).
 * sf_dense_ffn_fwd/bwd: the same equations with no pruning; fwd_ctx holds y1 (bf16 [T,F]).
 */
SF_API int sf_ffn_workspace_size(const sf_ffn_desc* desc, size_t* fwd_ctx_bytes, size_t* workspace_bytes);
SF_API int sf_sparse_ffn_fwd(const sf_ffn_desc* desc, const void* X, const void* W1, const void* W2,
                      void* Y, void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes,
                      void* stream);
SF_API int sf_sparse_ffn_bwd(const sf_ffn_desc* desc, const void* dY, const void* X, const void* W1,
                      const void* W2, const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2,
                      void* workspace, size_t workspace_bytes, void* stream);
SF_API int sf_dense_ffn_fwd(const sf_ffn_desc* desc, const void* X, const void* W1, const void* W2,
                     void* Y, void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes,
                     void* stream);
SF_API int sf_dense_ffn_bwd(const sf_ffn_desc* desc, const void* dY, const void* X, const void* W1,
                     const void* W2, const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Views into a sparse forward context (device pointers into fwd_ctx; nothing is copied). */
typedef enum sf_ctx_field {
  SF_CTX_Y2_VALS = 0,   /* bf16 [T, 2F/M] */
  SF_CTX_RELU_VALS = 1, /* bf16 [T, 2F/M] */
  SF_CTX_META = 2,      /* uint16 [T, F/(4M)] canonical */
  SF_CTX_COLIDX = 3,    /* uint8 [T/V, F/M, 4] */
  SF_CTX_Y1 = 4,        /* bf16 [T, F] (only with flags bit0) */
  SF_CTX_DY1_VALS = 5,  /* bf16 [T, 2F/M], lives in the WORKSPACE after sf_sparse_ffn_bwd; M != 8 only (for
                           M == 8 dy1 exists in its 2:4 form only, SF_CTX_DY1_VALS24) */
  SF_CTX_Y2_VALS24 = 6, /* bf16 [T, F/2]: y2 as a plain 2:4 operand over all F columns (M <= 8 only,
                           else SF_ERR_UNSUPPORTED): two stored values per four columns, explicit
                           zeros where a half-group keeps fewer than two */
  SF_CTX_Y2_META24 = 7, /* uint16 [T, F/16] canonical metadata of that operand (M <= 8 only) */
  SF_CTX_DY1_VALS24 = 8, /* bf16 [T, F/2]: dy1 at the positions of SF_CTX_Y2_META24; lives in the WORKSPACE
                           after sf_sparse_ffn_bwd (M <= 8 only) */
  SF_CTX_RELU_VALS24 = 9 /* bf16 [T, F/2]: ReLU(y1) at the positions of SF_CTX_Y2_META24 (M == 8 only) */
} sf_ctx_field;
SF_API int sf_ctx_view(const sf_ffn_desc* desc, const void* fwd_ctx_or_workspace, int field,
                const void** ptr, size_t* bytes);

/* One whole training step from HOST buffers (pinned memory is needed for the copies to overlap):
 * uploads X, W1, W2, dY into `device_staging`, runs sf_sparse_ffn_fwd + sf_sparse_ffn_bwd
 * (dense != 0: the dense pair) on `stream`, and downloads Y, dX, dW2, dW1. Uploads run on a
 * library-owned copy stream in the order X, W1, W2, dY, and each kernel waits only for the
 * operands it reads (the W1 prune and the y1 product start while W2 and dY are still in flight);
 * downloads run on a second copy stream, each as soon as its product is complete. Work already
 * on `stream` is ordered before the first upload, and `stream` is complete only after the last
 * download, so a cudaStreamSynchronize(stream) covers the whole step. Does not synchronise the
 * host. The two copy streams and nine events are created once per device on the first call (make
 * that call before any stream capture); calls on one device must not overlap on the host.
 * host_* pointers are HOST pointers; `device_staging` is a DEVICE buffer of
 * sf_ffn_host_staging_size() bytes. */
SF_API int sf_ffn_host_staging_size(const sf_ffn_desc* desc, size_t* bytes);
SF_API int sf_ffn_step_host(const sf_ffn_desc* desc, int dense, const void* host_X, const void* host_W1,
                     const void* host_W2, const void* host_dY, void* host_Y, void* host_dX,
                     void* host_dW1, void* host_dW2, void* device_staging, void* fwd_ctx,
                     size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * Sparse/dense step schedule (Section 5.3.2) and speed-up arithmetic (Sections 3.1 and 5.1).
 * Host-side logic; nothing here touches the GPU except the two dispatchers.
 *
 * A run of `total_steps` steps (0-based index) is: `warmup_steps` dense steps (the paper starts
 * V:N:M sparsification only after a dense warm-up, 1000 steps there), then `sparse_steps` sparse
 * steps, then dense steps to the end (sparse first, dense afterwards to recover accuracy).
 * SF_ERR_SHAPE when a count is negative, total_steps <= 0, the two phases exceed the run, or
 * `step` lies outside [0, total_steps).
 *
 * sf_schedule_speedup:    time of total_steps dense steps / time of the mixed schedule when a
 *                         sparse step is `sparse_step_speedup` times faster than a dense one
 *                         (Section 5.1's example: 2.2x on half of the steps -> 1.37x).
 * sf_ffn_flop_fraction:   FFN share of the training FLOPs, 18DF / (6(3DF + 2D(Nq + Nkv)H))
 *                         (Section 3.1).
 * sf_end_to_end_speedup:  1 / ((1 - f) + f / s): the whole-model effect of an s-times faster
 *                         FFN whose share of the time is f (Section 3.1 takes the FLOP share as
 *                         the time share).
 * sf_ffn_fwd_scheduled /  run the forward / backward step of the kind the schedule assigns to
 * sf_ffn_bwd_scheduled:   `step`; arguments as sf_sparse_ffn_fwd/bwd. Context and workspace of
 *                         sf_ffn_workspace_size() fit both kinds. Call both with the same step. */
typedef struct sf_schedule {
  int64_t warmup_steps;
  int64_t sparse_steps;
  int64_t total_steps;
} sf_schedule;
typedef enum sf_step_kind { SF_STEP_DENSE = 0, SF_STEP_SPARSE = 1 } sf_step_kind;
SF_API int sf_schedule_step_kind(const sf_schedule* schedule, int64_t step, int* kind);
SF_API int sf_schedule_speedup(const sf_schedule* schedule, double sparse_step_speedup, double* speedup);
SF_API int sf_ffn_flop_fraction(int64_t D, int64_t F, int64_t n_q_heads, int64_t n_kv_heads, int64_t head_dim,
                         double* fraction);
SF_API int sf_end_to_end_speedup(double ffn_fraction, double ffn_speedup, double* speedup);
SF_API int sf_ffn_fwd_scheduled(const sf_schedule* schedule, int64_t step, const sf_ffn_desc* desc,
                         const void* X, const void* W1, const void* W2, void* Y, void* fwd_ctx,
                         size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes, void* stream);
SF_API int sf_ffn_bwd_scheduled(const sf_schedule* schedule, int64_t step, const sf_ffn_desc* desc,
                         const void* dY, const void* X, const void* W1, const void* W2,
                         const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2,
                         void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------
 * The routed step: neuron-level experts that produce the V:N:M pattern (Section 3.1, Algorithm 3
 * "Convert Activation to Venom", Figure 4; Section 3.2.2 steps 1-3; Algorithm 1 line 6 `MoEToVenom`).
 *
 * Offline, the hidden features are clustered into E non-overlapping experts of Fe = F / E features
 * each and renumbered expert-major (rows of W1 and columns of W2 together: a reparametrisation of
 * the layer), so that expert e owns features [e Fe, (e+1) Fe); `means` holds the E cluster centres
 * as bf16 [E, D]. V:N:M keeps four of every M columns, hence E = M / 4 (M = 64: sixteen experts).
 * Per step each token goes to the expert with the largest x . mean (top-1, ties to the lower
 * expert; float32 accumulation), tokens are grouped by expert, and every product touches only the
 * token's expert block: y1, y2 = 2:4(ReLU(y1)^2) inside every four features of the block (greedy
 * magnitude rule of Section 2.3), Y = y2 W2^T, and Algorithm 2 on that mask. Interleaving the
 * expert blocks four features at a time gives the V:N:M matrix of Section 2.3 with the expert's
 * columns 4e..4e+3 kept in every group. Each product costs 1 / E of its dense counterpart (the
 * 2:4 ones half of that again); the token grouping is one gather pass per operand.
 *
 * Shape rules: T, D multiples of 256; 1 <= E <= 16; F / E a multiple of 256; T <= 2^20.
 * flags: SF_FFN_SAVE_Y1 only. Buffers as for the step above (sizes from
 * sf_routed_ffn_workspace_size; first 256 bytes of the workspace = status word).
 *
 * sf_router_route:   expert int32 [T] (and, optionally, logits float32 [T, E]) for X [T, D].
 * sf_routed_ffn_fwd: `forced_expert` (optional DEVICE int32 [T]) replaces the routing decision, for
 *                    stage-wise comparison with an implementation that accumulates the logits
 *                    differently; NULL = route with `means`.
 * sf_routed_ctx_view: device pointers into the context / workspace. Rows of the row-indexed fields
 *                    follow the grouped token order: SF_RCTX_SRC_OF_ROW gives the token of a row (-1 on
 *                    padding rows, which hold zeros), SF_RCTX_ROW_OF_TOKEN the inverse,
 *                    SF_RCTX_SEGMENTS = int32 [2E + 1]: first row of each expert's segment, total rows,
 *                    then the token count of each expert.
 */
typedef struct sf_router_desc {
  int64_t T, D, F;
  int32_t E;
  int32_t prune_mode;  /* as sf_ffn_desc */
  int32_t flags;       /* SF_FFN_SAVE_Y1 or 0 */
  int32_t reserved;
} sf_router_desc;
typedef enum sf_routed_ctx_field {
  SF_RCTX_EXPERT = 0,       /* int32 [T] */
  SF_RCTX_ROW_OF_TOKEN = 1, /* int32 [T] */
  SF_RCTX_SRC_OF_ROW = 2,   /* int32 [rows_max], rows_max = T + 256 E rounded up to 256 */
  SF_RCTX_SEGMENTS = 3,     /* int32 [2E + 1] */
  SF_RCTX_LOGITS = 4,       /* float32 [T, E] (written when the step routes itself) */
  SF_RCTX_Y2_VALS = 5,      /* bf16 [rows_max, Fe/2]: kept activations, two per four features of the expert block */
  SF_RCTX_RELU_VALS = 6,    /* bf16 [rows_max, Fe/2]: ReLU(y1) at the same positions */
  SF_RCTX_META = 7,         /* uint16 [rows_max, Fe/16]: canonical 2:4 metadata of those positions */
  SF_RCTX_Y1 = 8,           /* bf16 [rows_max, Fe] (only with SF_FFN_SAVE_Y1) */
  SF_RCTX_DY1_VALS = 9      /* bf16 [rows_max, Fe/2], in the WORKSPACE after sf_routed_ffn_bwd */
} sf_routed_ctx_field;
/* Offline clustering (HOST routine, all pointers are HOST pointers; no GPU is touched): balanced k-means
 * with L2 distance over the F feature vectors of W1 [F, D] (Figure 4a), at most `iters` Lloyd iterations.
 * Outputs: host_expert int32 [F] (expert of each feature, exactly F / E per expert), host_perm int32 [F]
 * (feature perm[i] of the old numbering becomes feature i of the expert-major one: apply it to the rows of
 * W1 and the columns of W2 once), host_means bf16 [E, D] (cluster centres = the router's ExpertMeans).
 * Deterministic. F % E == 0, 1 <= E <= 16. */
SF_API int sf_router_fit_host(const void* host_W1, int64_t F, int64_t D, int E, int iters, void* host_expert,
                              void* host_perm, void* host_means);
SF_API int sf_router_route(const void* X, const void* means, int64_t T, int64_t D, int E, void* expert,
                           void* logits, void* stream);
SF_API int sf_routed_ffn_workspace_size(const sf_router_desc* desc, size_t* fwd_ctx_bytes, size_t* workspace_bytes);
SF_API int sf_routed_ffn_fwd(const sf_router_desc* desc, const void* X, const void* W1, const void* W2,
                             const void* means, const void* forced_expert, void* Y, void* fwd_ctx,
                             size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes, void* stream);
SF_API int sf_routed_ffn_bwd(const sf_router_desc* desc, const void* dY, const void* X, const void* W1,
                             const void* W2, const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1,
                             void* dW2, void* workspace, size_t workspace_bytes, void* stream);
SF_API int sf_routed_ctx_view(const sf_router_desc* desc, const void* fwd_ctx_or_workspace, int field,
                              const void** ptr, size_t* bytes);

/* Bounded-wait self-test (the paper has no counterpart). Every device-side wait of the tensor-core
 * kernels gives up after a clock budget, raises the status word at the start of the workspace and
 * lets its CTA leave; sf_check_status then reports SF_ERR_TIMEOUT. This call runs that mechanism
 * in isolation: one CTA of one warp waits, with the same wait routine and a budget of
 * `budget_clocks` SM clocks (1 <= budget_clocks <= 2^31), on an mbarrier that nothing completes.
 * The wait runs out by construction, the kernel sets the status word and returns; nothing is
 * left waiting and the context stays usable. `workspace`: device buffer whose first int is the
 * (zeroed) status word. Enqueues on `stream`. */
SF_API int sf_selftest_wait_expiry(void* workspace, int64_t budget_clocks, void* stream);

/* Stage tracing, a measurement aid (the paper has no counterpart). `events` is a caller-owned HOST
 * array of `capacity` cudaEvent_t handles (created with timing enabled) that must stay valid until
 * tracing is switched off with capacity 0. While set, every FFN step call records one event
 * before its first kernel and one after each kernel, in launch order, on the call's stream:
 *   sparse fwd: 6 events (prune W1 | y1 product | V:N:M | W2 transpose | y3 product); intervals of
 *               kernels a path does not launch are empty (M <= 8: no W2 transpose; M == 8 with the
 *               selection fused into the y1 product: no V:N:M kernel)
 *   sparse bwd: 7 events (prune W2 | dy1 product | pack | dX product | dW2 product | dW1 product);
 *               for M <= 8 the dy1 product packs its own output and the pack interval is empty
 *   dense fwd: 3 events, dense bwd: 5 events.
 *   routed fwd: 6 events (prune W1 | route | group + tile tables + gather X | y1 product | y3 product)
 *   routed bwd: 7 events (prune W2 | gather dY | dy1 product | dX product | dW2 product | dW1 product).
 * sf_trace_count returns how many events have been recorded since sf_trace_set. Not thread-safe. */
SF_API int sf_trace_set(void** events, int capacity);
SF_API int sf_trace_count(void);

/* Synchronises `stream` and reads the device status word kept at the start of `workspace`:
 * SF_OK, or SF_ERR_TIMEOUT (once; the word is cleared) if a bounded wait inside a tensor-core
 * kernel expired. workspace == NULL names the status word of sf_gemm_sparse24_noalloc's built-in
 * scratch array on the current device. */
SF_API int sf_check_status(void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPARSEFFN_H_ */
