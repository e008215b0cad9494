/*
 * fblayout.h -- C ABI of the B200 attention-layer training step on one unified tiled layout.
 *
 * One transformer attention layer (pre-norm LayerNorm/RMSNorm, Q/K/V/O projections, causal or
 * full softmax attention with optional grouped-query heads), forward and backward, where every
 * matrix lives in a single reduction-aware tiled layout ("R-Tile", the paper's section 4.2) in
 * both passes.  The transposes the backward needs (W^T, X^T, head split/merge) are tile-index
 * remaps or operand-orientation flags of the tensor-core descriptors (the paper's section 4.3,
 * Eq. 3 and Eq. 4), never copies.
 *
 * Conventions that hold for every call
 *   - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are ordinary
 *     host memory.  The library allocates no device memory, never synchronises the device and
 *     enqueues all work on the CUDA stream handle passed as `stream` (a cudaStream_t cast to void*).
 *   - Matrices are in the storage dtype of the plan (fp32 or bf16) in R-Tile order and have
 *     exactly fbl_tensor_bytes() bytes; they must be 1024-byte aligned.  Vectors (gamma, beta,
 *     biases and their gradients) are plain fp32 arrays in both dtypes.
 *   - Padding slots of input matrices must hold zero (fbl_pack guarantees it); padding slots of
 *     output matrices are written as zero.
 *   - Gradients are overwritten, not accumulated.
 *   - Return value: FBL_OK (0) or a negative fbl_status.  Nothing throws, aborts or traps.  There is
 *     no CPU or library fallback: a shape the kernels cannot run is refused by fbl_plan_create.
 *
 * R-Tile, as laid out here (section 4.2: tile shape, intra-tile mapping Eq. 1, inter-tile mapping).
 *   A matrix [R, C] with e-byte elements is cut into storage tiles of tile_h = 8 rows by
 *   tile_w = 128/e columns (64 for bf16, 32 for fp32): one tile is 1 KiB, eight 128-byte rows,
 *   row-major inside (the paper's "horizontal strips" case tile_w <= C_w, with C_w one 128-byte
 *   line).  Tiles are ordered with the row-tile index fastest (the token axis is the dimension
 *   with more tile traversals): tile (tr, tc) is tile number tc * (R_pad/8) + tr.  Hence
 *       offset(r, c) = ((c / tile_w) * R_pad + r) * tile_w + c % tile_w          (in elements)
 *   with R_pad = R rounded up to 8 and C a multiple of tile_w.  Token matrices [B, T, C] use row
 *   r = b * T_pad + t with T_pad = T rounded up to 8, so every sequence starts on a tile boundary.
 */
#ifndef FBLAYOUT_H_
#define FBLAYOUT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FBL_OK = 0,
  FBL_ERR_INVALID_ARG = -1,
  FBL_ERR_UNSUPPORTED_SHAPE = -2,
  FBL_ERR_MISALIGNED = -3,
  FBL_ERR_WORKSPACE_TOO_SMALL = -4,
  FBL_ERR_CUDA = -5,
  FBL_ERR_TIMEOUT = -6
} fbl_status;

enum { FBL_DTYPE_FP32 = 0, FBL_DTYPE_BF16 = 1 };
enum { FBL_NORM_LAYERNORM = 0, FBL_NORM_RMSNORM = 1 };

/* The fine-tuning problem's shapes and flags (the paper's motivating example: one attention
 * block whose forward tensors are reused by the backward). */
typedef struct {
  int32_t batch, seq, d_model, n_q_heads, n_kv_heads, head_dim; /* GQA group = n_q_heads / n_kv_heads */
  int32_t dtype;        /* FBL_DTYPE_*  */
  int32_t norm;         /* FBL_NORM_*   */
  int32_t causal;       /* 0 / 1 */
  int32_t has_bias;     /* 0 / 1: biases on Q, K, V and O projections */
  int32_t residual;     /* 0 / 1: Y = X + attention(norm(X)) */
  float eps;
  float softmax_scale;  /* <= 0 selects 1/sqrt(head_dim) */
} fbl_layer_desc;

/* Tensor ids for fbl_tensor_bytes, fbl_tile_offset, fbl_pack and fbl_unpack.  The *_HEADS ids are
 * index-map views [B, H, T, head_dim] of the same buffers as Q, K, V and A (no data moves). */
enum {
  FBL_T_X = 0, FBL_T_Y, FBL_T_DY, FBL_T_DX,          /* [B, T, D]               */
  FBL_T_WQ, FBL_T_WK, FBL_T_WV, FBL_T_WO,            /* [D,Dq] [D,Dkv] [D,Dkv] [Dq,D] (and their gradients) */
  FBL_T_XN, FBL_T_Q, FBL_T_K, FBL_T_V, FBL_T_A,      /* [B, T, D | Dq | Dkv | Dkv | Dq] */
  FBL_T_Q_HEADS, FBL_T_K_HEADS, FBL_T_V_HEADS, FBL_T_A_HEADS, /* [B, H, T, hd] views */
  FBL_T_WQ_T, FBL_T_WK_T, FBL_T_WV_T, FBL_T_WO_T,    /* transposed views [C, R] of the weights */
  FBL_T_MEM, FBL_T_DMEM,                             /* cross-attention plans only: memory [B, Tkv, Dmem] and its gradient */
  FBL_T_COUNT
};

/* Tile maps f of Eq. 3 (row-major tile numbering of the source view -> of the destination view). */
enum {
  FBL_MAP_SPLIT_Q = 0,   /* [B*T_pad, Dq] flat view  -> [B, Hq, T_pad, hd] head view (reshape o transpose) */
  FBL_MAP_MERGE_Q,       /* inverse                                                                   */
  FBL_MAP_SPLIT_KV,      /* same for Dkv / Hkv                                                        */
  FBL_MAP_MERGE_KV,
  FBL_MAP_TRANSPOSE_WQ,  /* [D, Dq] -> [Dq, D] */
  FBL_MAP_TRANSPOSE_WO,  /* [Dq, D] -> [D, Dq] */
  FBL_MAP_PHYS_Q,        /* flat-view tile number -> physical tile slot in memory (inter-tile mapping) */
  FBL_MAP_PHYS_WQ,
  FBL_MAP_COUNT
};

typedef struct fbl_plan fbl_plan; /* opaque: padded sizes, index-map constants, kernel choices.  Enqueue calls on
                                   * one plan keep a little bookkeeping in it: use one plan per host thread. */

/* Host code only (no device work; it asks the runtime for the current device's SM count to size grids and work
 * areas, and plans for 148 SMs when there is no device).  Validates the description against the tile-propagation legality checks of section 4.3
 * (head_dim and d_model multiples of tile_w, n_q_heads a multiple of n_kv_heads) and the kernels'
 * limits, then builds the plan.  *out is owned by the caller; release with fbl_plan_destroy.
 * The plan also fixes, from the shapes alone, into how many slices the token-axis reductions of the weight
 * gradients are cut (1 for all but layers with few weight tiles and many tokens).  Environment variables
 * read here, for tuning and tests only: FBL_KSPLIT_O and FBL_KSPLIT_QKV override those slice counts,
 * FBL_VERBOSE prints the ones chosen to stderr.  Three more, again for tuning and tests only: FBL_GEMM_PAIR (0: never use the CTA-pair GEMM kernel, 1: use it wherever its tile shape is
 * legal; unset: large launches only), FBL_GEMM_ESETS (1 or 2 sets of epilogue warps in the single-CTA GEMM kernel;
 * unset: 2 where every block of the launch has one tile) and FBL_FWD_TILES (1 or 2 query tiles per
 * forward-attention block at head_dim 64; unset: by sequence length). */
int fbl_plan_create(const fbl_layer_desc* desc, fbl_plan** out);
void fbl_plan_destroy(fbl_plan* plan);

/* Padded R-Tile size in bytes of a matrix (physical ids only; views return the size of their buffer).  Rows are
 * padded to whole tiles only (seq and weight rows rounded up to tile_h = 8), which keeps the padded share far
 * inside the 10 % limit of the paper's tile-selection constraint C3 (section 4.2, candidate generation). */
int fbl_tensor_bytes(const fbl_plan* plan, int tensor_id, size_t* bytes);

/* Sizes of the three caller-owned work areas: `saved` carries forward tensors into the backward
 * (the E_reuse edges of the paper's graph, section 3.1: norm statistics, Xn, Q, K, V, A, LSE);
 * the scratch areas hold per-call temporaries. */
int fbl_workspace_bytes(const fbl_plan* plan, size_t* saved, size_t* scratch_fwd, size_t* scratch_bwd);

/* Where the step's intermediates live inside the caller's work areas (byte offset and size), so that a caller
 * can inspect them after synchronising: matrices are R-Tile buffers readable with fbl_unpack under the tensor id
 * of the same shape (XN; Q for Q, A, dA, dQ; K for K, V, dK, dV); STATS is fp32 [B*T_pad][2] = (mean, rstd);
 * LSE and D are fp32 [B][Hq][T_pad].  FBL_WS_STATS .. FBL_WS_LSE are offsets into `saved` (section 3.1's reused
 * forward tensors), the others into the backward scratch. */
enum {
  FBL_WS_STATS = 0, FBL_WS_XN, FBL_WS_Q, FBL_WS_K, FBL_WS_V, FBL_WS_A, FBL_WS_LSE,
  FBL_WS_D, FBL_WS_DA, FBL_WS_DQ, FBL_WS_DK, FBL_WS_DV, FBL_WS_DXN,
  FBL_WS_PARTIALS,   /* partial sums of the backward's token-axis reductions (bias column sums, dgamma / dbeta) */
  FBL_WS_COUNT
};
int fbl_workspace_offset(const fbl_plan* plan, int what, size_t* offset, size_t* bytes);

/* Element map (pure host integer code): logical index -> element offset in the R-Tile buffer, i.e. the
 * composition of section 4.2's inter-tile mapping (which tile, row-tile index fastest) and intra-tile mapping
 * (row-major inside the 8 x tile_w tile).
 * idx is [b, t, c, 0] for token matrices, [r, c, 0, 0] for weights and transposed views,
 * [b, h, t, d] for head views.  Returns < 0 if idx is out of range. */
int64_t fbl_tile_offset(const fbl_plan* plan, int tensor_id, const int32_t idx[4]);

/* Tile map f of Eq. 3, composed and strength-reduced as in Eq. 4 (host integer code). */
int fbl_tile_map(const fbl_plan* plan, int map_id, int64_t src_tile, int64_t* dst_tile);

/* Layout conversion at the graph boundary only (row-major dense <-> R-Tile), device to device: section 4.4 keeps
 * one layout inside the graph and converts only where tensors enter or leave it.  Never part of a training step. */
int fbl_pack(const fbl_plan* plan, int tensor_id, const void* rowmajor_dev, void* tiled_dev, void* stream);
int fbl_unpack(const fbl_plan* plan, int tensor_id, const void* tiled_dev, void* rowmajor_dev, void* stream);

/* Forward of the attention block of the paper's motivating example (section 2: projections, P = softmax(Q K^T),
 * O = P V, output projection): Y = [X +] softmax-attention(norm(X)) Wo [+ bo].  Fills `saved`, the forward
 * tensors the backward reuses (the E_reuse edges of section 3.1), in the same layout the backward reads them in.
 * Biases and beta may be NULL when the plan has none.  The call first clears the status word at the start of
 * `scratch` (see fbl_status_poll). */
int fbl_layer_fwd(const fbl_plan* plan, const void* X, const float* gamma, const float* beta,
                  const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                  const float* bq, const float* bk, const float* bv, const float* bo,
                  void* Y, void* saved, void* scratch, void* stream);

/* Backward of the same block (section 2's gradient operators; section 3.2's reduce-axis conflicts are resolved by
 * operand orientation, not by copies): every gradient of sum(Y * dY).  Matrix gradients are in the storage dtype
 * in R-Tile order; vector gradients are fp32.  db* may be NULL when the plan has no biases, dbeta for RMSNorm.
 * The call first clears the status word at the start of its own `scratch`: a caller that wants to see a
 * forward-pass time-out after the backward has been enqueued gives the two passes separate scratch buffers
 * (scratch_fwd_bytes / scratch_bwd_bytes) and polls both. */
int fbl_layer_bwd(const fbl_plan* plan, const void* dY, const void* X, const float* gamma,
                  const void* Wq, const void* Wk, const void* Wv, const void* Wo, const void* saved,
                  void* dX, void* dWq, void* dWk, void* dWv, void* dWo,
                  float* dbq, float* dbk, float* dbv, float* dbo, float* dgamma, float* dbeta,
                  void* scratch, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * The feed-forward half of the block on the same layout: pre-norm, up projection (plus a gate projection for the
 * gated variant), activation, down projection, optional residual.  Its matmuls are the paper's reduce-axis-conflict
 * operator (section 4.1: Y = X W reduces over d_in, dW = X^T dY over the tokens, dX = dY W^T over d_out) at the
 * shapes of its single-MatMul benchmark (section 5.2, R-Tile ablation: forward (512, 2048, 8192), backward
 * (512, 8192, 2048)); as in the attention layer every operand stays in R-Tile order in both passes and W^T, Xn^T,
 * H^T are operand-orientation flags, never copies.
 *   forward   Xn = norm(X); U = Xn W1 + b1; [G = Xn Wg + bg;]  H = gelu(U) | silu(G) * U;  Y = H W2 + b2 [+ X]
 *   backward  dW2 = H^T dY, db2; dH = dY W2^T; dU = dH gelu'(U) | dU = dH silu(G), dG = dH U silu'(G);
 *             dW1 = Xn^T dU, db1 [, dWg = Xn^T dG, dbg]; dXn = dU W1^T [+ dG Wg^T]; norm backward -> dX, dgamma, dbeta
 * gelu is the tanh form u/2 (1 + tanh(sqrt(2/pi) (u + 0.044715 u^3))).  Conventions (pointers, alignment, padding,
 * status word, return codes) are those of the attention layer's calls.  W1, Wg: [d_model, d_ff]; W2: [d_ff, d_model];
 * b1, bg: [d_ff]; b2: [d_model].  Wg, bg, dWg, dbg are NULL for FBL_ACT_GELU; biases and their gradients NULL without
 * has_bias; beta, dbeta NULL for RMSNorm. */
enum { FBL_ACT_GELU = 0, FBL_ACT_SWIGLU = 1 };
typedef struct {
  int32_t batch, seq, d_model, d_ff;
  int32_t dtype;        /* FBL_DTYPE_*  */
  int32_t norm;         /* FBL_NORM_*   */
  int32_t act;          /* FBL_ACT_*    */
  int32_t has_bias;     /* 0 / 1 */
  int32_t residual;     /* 0 / 1: Y = X + mlp(norm(X)) */
  float eps;
} fbl_mlp_desc;
typedef struct fbl_mlp_plan fbl_mlp_plan;
/* Matrix ids for fbl_mlp_tensor_bytes, fbl_mlp_pack and fbl_mlp_unpack. */
enum { FBL_MT_X = 0 /* [B, T, d_model]: X, Y, dY, dX, Xn, dXn */, FBL_MT_H /* [B, T, d_ff]: U, G, H, dU, dG */,
       FBL_MT_W1 /* [d_model, d_ff]: W1, Wg and gradients */, FBL_MT_W2 /* [d_ff, d_model] */, FBL_MT_COUNT };
/* Offsets of the block's intermediates: STATS .. H inside `saved`, the others inside the backward scratch. */
enum { FBL_MWS_STATS = 0, FBL_MWS_XN, FBL_MWS_U, FBL_MWS_G, FBL_MWS_H, FBL_MWS_DU, FBL_MWS_DG, FBL_MWS_DXN, FBL_MWS_COUNT };

int fbl_mlp_plan_create(const fbl_mlp_desc* desc, fbl_mlp_plan** out);   /* d_model, d_ff multiples of tile_w */
void fbl_mlp_plan_destroy(fbl_mlp_plan* plan);
int fbl_mlp_tensor_bytes(const fbl_mlp_plan* plan, int matrix_id, size_t* bytes);
int fbl_mlp_workspace_bytes(const fbl_mlp_plan* plan, size_t* saved, size_t* scratch_fwd, size_t* scratch_bwd);
int fbl_mlp_workspace_offset(const fbl_mlp_plan* plan, int what, size_t* offset, size_t* bytes);
int fbl_mlp_pack(const fbl_mlp_plan* plan, int matrix_id, const void* rowmajor_dev, void* tiled_dev, void* stream);
int fbl_mlp_unpack(const fbl_mlp_plan* plan, int matrix_id, const void* tiled_dev, void* rowmajor_dev, void* stream);
int fbl_mlp_fwd(const fbl_mlp_plan* plan, const void* X, const float* gamma, const float* beta,
                const void* W1, const void* Wg, const void* W2, const float* b1, const float* bg, const float* b2,
                void* Y, void* saved, void* scratch, void* stream);
int fbl_mlp_bwd(const fbl_mlp_plan* plan, const void* dY, const void* X, const float* gamma,
                const void* W1, const void* Wg, const void* W2, const void* saved,
                void* dX, void* dW1, void* dWg, void* dW2, float* db1, float* dbg, float* db2,
                float* dgamma, float* dbeta, void* scratch, void* stream);
int fbl_mlp_status_poll(const fbl_mlp_plan* plan, const void* scratch, int32_t* device_status);
/* 0 = default kernels (tcgen05 for bf16), 1 = FFMA kernels only, as fbl_plan_set_kernel_path. */
int fbl_mlp_set_kernel_path(fbl_mlp_plan* plan, int path);
int64_t fbl_mlp_launch_count(const fbl_mlp_plan* plan);

/* ---------------------------------------------------------------------------------------------------------------
 * Low-rank adapters on the Q, K and V projections with the base weights frozen: the paper's fine-tuning setting
 * (section 2, motivating example X A_LoRA B_LoRA; section 5.1).  Q = Xn Wq + bq + (Xn Aq) Bq, likewise K and V; only
 * the adapters and the layer input receive gradients, so the weight-gradient products of the frozen projections
 * (and their token-axis reductions) are skipped, and the adapters add thin products whose reduction axes are the
 * rank (forward, dT B^T) and the tokens (dA = Xn^T dT, dB = T^T d*).  A scale alpha / r is folded into B by the
 * caller.
 *
 * Storage.  The three adapters live in two R-Tile matrices with each adapter's rank padded to one 64-wide block
 * (FBL_LORA_BLOCK) of zeros, so that every product is whole tiles:
 *   A_all [d_model, 192]              column block i (i = 0 q, 1 k, 2 v) holds A_i in its first `rank` columns;
 *   B_all [192, d_q + 2 d_kv]         block-diagonal: rows 64 i .. 64 i + rank of column block i hold B_i, the rest 0.
 * fbl_lora_pack / fbl_lora_unpack convert one adapter matrix (row-major [d_model, rank] or [rank, d_out]) to and from
 * its block; the caller zero-fills A_all and B_all once before packing.  dA_all and dB_all come back in the same
 * shapes; off-diagonal blocks of dB_all are not gradients of anything and must be ignored (fbl_lora_unpack does).
 *
 * fbl_plan_enable_lora must precede fbl_workspace_bytes (the work areas grow by T = Xn A_all and dT).  rank 1..64.
 * Biases, if the plan has them, are applied but frozen; dgamma / dbeta may be NULL (frozen norm). */
enum { FBL_LORA_BLOCK = 64 };
enum { FBL_LORA_AQ = 0, FBL_LORA_AK, FBL_LORA_AV, FBL_LORA_BQ, FBL_LORA_BK, FBL_LORA_BV };
int fbl_plan_enable_lora(fbl_plan* plan, int rank);
int fbl_lora_bytes(const fbl_plan* plan, size_t* a_all_bytes, size_t* b_all_bytes);
int fbl_lora_pack(const fbl_plan* plan, int which, const void* rowmajor_dev, void* all_dev, void* stream);
int fbl_lora_unpack(const fbl_plan* plan, int which, const void* all_dev, void* rowmajor_dev, void* stream);
int fbl_layer_fwd_lora(const fbl_plan* plan, const void* X, const float* gamma, const float* beta,
                       const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                       const float* bq, const float* bk, const float* bv, const float* bo,
                       const void* A_all, const void* B_all, void* Y, void* saved, void* scratch, void* stream);
int fbl_layer_bwd_lora(const fbl_plan* plan, const void* dY, const void* X, const float* gamma,
                       const void* Wq, const void* Wk, const void* Wv, const void* Wo,
                       const void* A_all, const void* B_all, const void* saved,
                       void* dX, void* dA_all, void* dB_all, float* dgamma, float* dbeta, void* scratch, void* stream);

/* Token-axis column reduction used for every bias gradient (db = sum over tokens, the matmul
 * backward's M-axis reduction of section 4.1): out[c] = sum_r M[r, c] for an R-Tile matrix of
 * `rows` x `cols` (rows a multiple of 8, cols of tile_w) in the plan's dtype.  Two stages over tiles:
 * per-slab partial sums into `scratch` (fbl_colsum_scratch_bytes), then a tree over slabs. */
int fbl_colsum_scratch_bytes(const fbl_plan* plan, int64_t rows, int64_t cols, size_t* bytes);
int fbl_colsum(const fbl_plan* plan, const void* M_dev, int64_t rows, int64_t cols,
               float* out_dev, void* scratch_dev, void* stream);

/* (No counterpart in the paper.)  fbl_colsum for callers that cannot hand over scratch memory: code that runs
 * where device allocation is off limits -- inside a framework's allocator hook or out-of-memory handler, in a
 * plugin that was given fixed input and output buffers and nothing else, or on a path that must not disturb a
 * caching allocator.  The per-slab partial sums go to a fixed 1 MiB array that is part of the library image
 * (every GPU that loads the library carries it until the process exits), so this call allocates nothing, on the
 * host side of CUDA or through any library.  Same arguments and result as fbl_colsum minus `scratch_dev`.
 *   - Limit: ceil(rows / 256) * cols <= 262144 (for example 16384 rows x 4096 columns); beyond it the call
 *     returns FBL_ERR_WORKSPACE_TOO_SMALL and enqueues nothing.
 *   - The first call on each device looks up the array's device address (with that device current).  Make that
 *     first call at start-up, outside any stream capture and before memory is tight: with the runtime's lazy
 *     module loading it may be the call that loads the library image carrying the array onto the device, which
 *     the driver does with an allocation of its own; "allocates nothing" holds from the second call on.  The
 *     address is cached per device ordinal and does not survive a device reset.
 *   - All calls on a device share the one array.  Each call overwrites the part it uses before reading it, so
 *     earlier contents never leak into a result, but two calls that can run at the same time on the GPU (different
 *     streams, no ordering between them) race; order them. */
int fbl_colsum_noalloc(const fbl_plan* plan, const void* M_dev, int64_t rows, int64_t cols,
                       float* out_dev, void* stream);

/* After the caller has synchronised the stream: reads back the device status word kept at the start
 * of `scratch` (set when a bounded wait inside a kernel expired).  Synchronous 4-byte copy. */
int fbl_status_poll(const fbl_plan* plan, const void* scratch, int32_t* device_status);

/* Self-test of the failure detection (no counterpart in the paper).  Every wait inside the tensor-core kernels is
 * bounded: when it expires, the kernel records a code in the status word at the start of `scratch`, leaves its
 * loops, releases its tensor memory and returns, so the context stays usable.  This call enqueues one tiny kernel
 * that waits, through the same code, on a barrier nothing will ever signal, with `limit_cycles` clock cycles as
 * the bound (clamped to [1e3, 2e9]); it first zeroes the first 8 bytes of `scratch` (1024-byte aligned device
 * memory, at least 8 bytes).  After the caller has synchronised, fbl_status_poll on that buffer returns
 * FBL_ERR_TIMEOUT with *device_status == 901, and the int32 behind the status word holds 1 (the block ran to its
 * normal end). */
int fbl_selftest_wait_timeout(void* scratch, int64_t limit_cycles, void* stream);

/* ---------------------------------------------------------------------------------------------------------------
 * Offline tile selection (section 4.2, step 1 and Eq. 1, Eq. 2; Supplement Algorithm 1), restated for this GPU.
 *
 * fbl_rtile_candidates: storage-tile shape candidates for a set of matrices.  The initial pool is every
 * (tile_h, tile_w) with tile_h in {1, 2, 4, 8, 16, 32, 64, 128} rows and tile_w * elem_bytes in {32, 64, 128, 256,
 * 512} bytes; it is filtered by the three constraints in the paper's order and each survivor gets its N_cache of
 * Eq. 1 (with the 1 x 128-byte line of this memory system as the cache tile) and its worst padding ratio:
 *   C1 computation: a tile row must be exactly the 128-byte span of the tensor cores' swizzled shared-memory operand
 *      rows, and tile_h a multiple of the 8-row swizzle atom that still divides the 128-row compute tile (so that
 *      any run of tiles is a legal K-major or MN-major operand: the tile-invariance property);
 *   C2 memory: a tile is at most one 4 KiB bulk-copy box row group and starts on a 128-byte line (whole lines);
 *   C3 shape: the padded size of every matrix exceeds its size by at most `max_pad_ratio` (the paper uses 0.10).
 * `shapes` holds n_shapes pairs (rows, cols).  Survivors are written to `out` (at most max_out), ordered by
 * ascending N_cache, then ascending padding; the return value is their count (or a negative fbl_status).
 * reject_counts[0..2], if not NULL, receive how many pool entries C1, C2 and C3 removed. */
typedef struct { int32_t tile_h, tile_w, n_cache; float pad_ratio; } fbl_rtile_cand;
int fbl_rtile_candidates(const int64_t* shapes, int n_shapes, int elem_bytes, float max_pad_ratio,
                         fbl_rtile_cand* out, int max_out, int32_t reject_counts[3]);

/* The compute-tile configuration of one GEMM launch of the step, as chosen offline (the profiling step of
 * section 4.2 / 6 and the argmax of Eq. 2 live in the Python module rtile.py, which times the candidates through
 * these calls): output-tile width 128 or 256 (0: built-in heuristic), CTA-pair kernel 0 / 1 (-1: heuristic),
 * epilogue warp sets 1 / 2 (0: heuristic).  A choice whose tile shape is not legal for the launch's shapes falls
 * back to the heuristic.  Takes effect for later fbl_layer_fwd / fbl_layer_bwd calls on this plan. */
enum { FBL_GEMM_PROJ_QKV = 0, FBL_GEMM_PROJ_O, FBL_GEMM_DWO_DA, FBL_GEMM_DWQKV_DXN, FBL_GEMM_LAUNCH_COUNT };
int fbl_plan_set_gemm_choice(fbl_plan* plan, int launch_id, int tile_n, int cta_pair, int epilogue_sets);

/* ---------------------------------------------------------------------------------------------------------------
 * Tile propagation and index-transformation elimination for an arbitrary chain of reshape / permute operators
 * (section 4.3: the three dependency checks, Eq. 3 T_dst[i] = f(T_src[j]), Eq. 4 f = f_n o ... o f_1 and the strength
 * reduction of the composed index function).  Pure host integer code.
 *
 * A tensor of logical shape `shape` (rank <= 8, row-major) is stored as the R-Tile matrix [prod(shape[:-1]), shape[-1]]
 * with tile_h x tile_w tiles.  After the chain the result, of whatever rank, is stored the same way with the same
 * tile shape.  If the chain only moves whole tiles, fbl_tile_chain_create builds the composed tile map f (source tile
 * number -> destination tile number, both row-major over their tile grids) as a short list of terms
 *     f(j) = sum_k ((j / div_k) % mod_k) * mul_k           (mod_k = 0: no modulo, the outermost digit)
 * in which digits that stay adjacent have been merged (the rule (i mod Ca) mod Cb = i mod Cb for Cb | Ca applied to
 * the whole chain), and returns FBL_OK.  Otherwise it returns FBL_ERR_UNSUPPORTED_SHAPE and reports the first
 * operator that breaks the tile structure and which check it fails:
 *   FBL_TP_DIMENSION   the axes a tile spans do not end up as the destination's tile axes (the chain moves the tile's
 *                      row or column axis elsewhere, e.g. a transpose of the last two axes, or changes the element
 *                      count: an expand / repeat, where the paper too falls back);
 *   FBL_TP_BOUNDARY    a reshape cuts inside a tile: the split (or merged) extent is not a whole number of tiles
 *                      (hidden 768 -> 16 x 48 with tile_w 64), or the innermost row extent is not a multiple of tile_h;
 *   FBL_TP_CONTINUITY  the elements of a tile row (or the rows of a tile) lose their stride-1 order.
 * Sizes must already include padding (a 197-token sequence is passed as 200 for tile_h = 8). */
enum { FBL_VIEW_RESHAPE = 0, FBL_VIEW_PERMUTE = 1, FBL_VIEW_EXPAND = 2 };
enum { FBL_TP_OK = 0, FBL_TP_DIMENSION = 1, FBL_TP_BOUNDARY = 2, FBL_TP_CONTINUITY = 3 };
typedef struct {
  int32_t kind;        /* FBL_VIEW_*                                                              */
  int32_t rank;        /* rank of the result                                                      */
  int64_t shape[8];    /* RESHAPE / EXPAND: the new shape                                          */
  int32_t perm[8];     /* PERMUTE: result axis k is input axis perm[k]                            */
} fbl_view_op;
typedef struct { int64_t div, mod, mul; } fbl_tile_term;
typedef struct fbl_tile_chain fbl_tile_chain;
int fbl_tile_chain_create(const int64_t* shape, int rank, int tile_h, int tile_w, const fbl_view_op* ops, int n_ops,
                          fbl_tile_chain** out, int32_t* failed_op, int32_t* failed_check);
void fbl_tile_chain_destroy(fbl_tile_chain* chain);
int64_t fbl_tile_chain_tiles(const fbl_tile_chain* chain);                       /* tiles of the tensor */
int fbl_tile_chain_terms(const fbl_tile_chain* chain, fbl_tile_term* terms, int max_terms);   /* returns the count */
int fbl_tile_chain_map(const fbl_tile_chain* chain, int64_t src_tile, int64_t* dst_tile);     /* evaluates f */

/* Rotary position embedding on Q and K (an element-wise, position-dependent rotation between the projections and the
 * scores: in the paper's classification a layout-independent operator, so it runs in place on the R-Tile buffers
 * without any conversion).  Half-split pairing: inside every head element i < head_dim/2 is paired with element
 * i + head_dim/2 and the pair of token t turns by t * base^(-2i/head_dim).  `saved` then holds the rotated Q and K;
 * the backward rotates dQ and dK by the opposite angle before the weight-gradient and input-gradient products.
 * base > 1 (10000 is customary); head_dim a multiple of 16.  Applies to fbl_layer_fwd / bwd and their _lora forms. */
int fbl_plan_enable_rope(fbl_plan* plan, float base);

/* ---------------------------------------------------------------------------------------------------------------
 * Cross-attention (section 2 names it beside MHA and GQA among the attention forms whose partitioning the layout has to
 * serve; Whisper and Stable Diffusion in the model table contain it).  The layer of fbl_layer_fwd with K and V
 * projected from a second sequence, the memory M [batch, seq_kv, d_mem], used as it is (no norm on it):
 *     Xn = norm(X);  Q = Xn Wq + bq;  K = M Wk + bk;  V = M Wv + bv;  A = softmax(scale Q K^T) V per head, no mask;
 *     Y = A Wo + bo (+ X).
 * The same kernels run it: the attention kernels take the key side's row count and sequence length separately from
 * the query side's, the projections of the two sides share one grouped launch, and the backward adds dM = dK Wk^T +
 * dV Wv^T (one accumulator, two reduction loops).  Nothing is transposed or re-partitioned for the second sequence.
 *
 * fbl_xattn_plan_create: desc describes the query side (seq = query tokens per sequence; causal must be 0); seq_kv >= 1
 * memory tokens per sequence; d_mem a multiple of tile_w.  The plan is an fbl_plan: fbl_tensor_bytes / fbl_pack /
 * fbl_unpack / fbl_tile_offset (K, V, Wk, Wv take the memory's extents; FBL_T_MEM / FBL_T_DMEM are valid),
 * fbl_workspace_bytes / _offset, fbl_status_poll, fbl_profile_* and fbl_plan_destroy apply.  fbl_layer_fwd / _bwd
 * reject it (FBL_ERR_INVALID_ARG) and fbl_xattn_fwd / _bwd reject a self-attention plan; adapters and the rotary
 * embedding are not available on it.
 * All pointers are device pointers, 1024-byte aligned, in the R-Tile layout; vectors fp32; ownership stays with the
 * caller; the calls enqueue on `stream` and return.  Errors as for fbl_layer_fwd / _bwd. */
int fbl_xattn_plan_create(const fbl_layer_desc* desc, int32_t seq_kv, int32_t d_mem, fbl_plan** out);
int fbl_xattn_fwd(const fbl_plan* plan, const void* X, const void* M, const float* gamma, const float* beta,
                  const void* Wq, const void* Wk, const void* Wv, const void* Wo, const float* bq, const float* bk,
                  const float* bv, const float* bo, void* Y, void* saved, void* scratch, void* stream);
/* Adds dM [batch, seq_kv, d_mem] to the outputs of fbl_layer_bwd; dWk, dWv are [d_mem, Dkv]. */
int fbl_xattn_bwd(const fbl_plan* plan, const void* dY, const void* X, const void* M, const float* gamma,
                  const void* Wq, const void* Wk, const void* Wv, const void* Wo, const void* saved, void* dX, void* dM,
                  void* dWq, void* dWk, void* dWv, void* dWo, float* dbq, float* dbk, float* dbv, float* dbo,
                  float* dgamma, float* dbeta, void* scratch, void* stream);

/* Kernel family used by later calls on this plan: 0 = default (tcgen05 tensor-core kernels for bf16
 * wherever one exists for the shape, FFMA kernels for fp32), 1 = FFMA kernels only (fp32 arithmetic on
 * the same layout; lets a caller cross-check the tensor-core path on the device). */
int fbl_plan_set_kernel_path(fbl_plan* plan, int path);

/* Optional per-step device timing.  fbl_profile_enable(plan, 1) creates CUDA events (host objects); while
 * enabled, fbl_layer_fwd / fbl_layer_bwd record one event after each of their steps.  After the caller has
 * synchronised, fbl_profile_read returns the number of steps of the most recent call and fills their names
 * (static strings) and durations in milliseconds.  fbl_launch_count is the number of kernels this plan
 * has enqueued since it was created. */
int fbl_profile_enable(fbl_plan* plan, int enable);
int fbl_profile_read(const fbl_plan* plan, int max_steps, const char** names, float* ms);
int64_t fbl_launch_count(const fbl_plan* plan);

const char* fbl_strerror(int status);
/* Text of the last CUDA runtime error seen by this thread inside the library ("" if none). */
const char* fbl_last_error_detail(void);

#ifdef __cplusplus
}
#endif
#endif /* FBLAYOUT_H_ */
