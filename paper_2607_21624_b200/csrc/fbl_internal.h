// Internal declarations shared by the translation units of libfblayout.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "fblayout.h"

#define FBL_TILE_H 8
#define FBL_ALIGN 1024
#define FBL_PROF_MAX 32

// ---------------------------------------------------------------------------------------------
// R-Tile element map (section 4.2).  Storage tile = 8 rows x 128 bytes, row-major inside; tiles
// ordered with the row-tile index fastest.  TW = elements per 128-byte tile row.
// ---------------------------------------------------------------------------------------------
template <int TW>
__host__ __device__ __forceinline__ int64_t rt_off(int64_t r_pad, int64_t r, int c) {
  return ((int64_t)(c / TW) * r_pad + r) * TW + (c % TW);
}
__host__ __device__ __forceinline__ int64_t rt_off_dyn(int tw, int64_t r_pad, int64_t r, int64_t c) {
  return ((c / tw) * r_pad + r) * tw + (c % tw);
}

template <typename T> struct tile_w_of { static constexpr int value = 128 / (int)sizeof(T); };

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct fbl_plan {
  fbl_layer_desc d;
  int e;        // bytes per element
  int tw;       // tile_w in elements
  int t_pad;    // seq rounded up to 8
  int64_t n_pad;  // batch * t_pad
  // Key side of the attention: the same sequence in self-attention; in a cross-attention plan (cross = 1) the memory
  // sequence [batch, seq_kv, d_mem] that K and V are projected from
  int cross, seq_kv, t_pad_kv, d_mem;
  int64_t n_pad_kv;
  int dq, dkv, group;
  float scale;
  int sm_count;
  int use_tc;   // 1: tensor-core (tcgen05) kernels where one exists for the shape; 0: FFMA kernels only
  // byte offsets inside `saved`
  size_t sv_stats, sv_xn, sv_q, sv_k, sv_v, sv_a, sv_lse, saved_bytes;
  // byte offsets inside the backward scratch
  size_t sb_da, sb_dvec, sb_dqacc, sb_dq, sb_dk, sb_dv, sb_dxn, sb_part, scratch_bwd_bytes;
  size_t scratch_fwd_bytes;
  size_t part_bytes;
  // reduction-loop slicing of the weight-gradient GEMMs (1: none) and their fp32 accumulation areas, which
  // follow the status word so that one fill zeroes both
  int ksplit_o, ksplit_qkv;
  size_t sb_acc_o, sb_acc_qkv, acc_bytes;
  // cross-attention only: slices of dWk / dWv, their accumulation area, dM's place is the caller's; partial sums of
  // the dK / dV column sums
  int ksplit_kv;
  size_t sb_acc_kv, sb_part_kv;
  size_t zero_bytes;        // leading part of the backward scratch that every step starts by zero-filling
  // tuning knobs, read from the environment once, at plan creation (0 / -1 = the library's own choice)
  int knob_gemm_pair;       // -1 by size, 0 never the CTA-pair GEMM kernel, 1 wherever its tile shape is legal
  int knob_gemm_esets;      // 0 by tiles per block, 1 / 2 sets of epilogue warps
  int knob_fwd_tiles;       // 0 by sequence length, 1 / 2 query tiles per forward-attention block at head_dim 64
  // low-rank adapters on Q, K, V (fbl_plan_enable_lora): rank, and the offsets of T = Xn [Aq|Ak|Av] inside `saved`,
  // of dT and of the unused norm-parameter gradients inside the backward scratch
  float rope_base;          // > 0: rotary position embedding on Q and K (fbl_plan_enable_rope)
  int lora_rank;
  size_t sv_t, sb_dt, sb_frozen;
  // Compute-tile configuration of each GEMM launch of a step, fixed offline by the tile chooser (0 / -1: the
  // built-in heuristics decide): output-tile width, CTA-pair kernel, sets of epilogue warps.
  struct GemmChoice { int bn, pair, esets; } choice[FBL_GEMM_LAUNCH_COUNT];
  // bookkeeping of the enqueue calls (they take the plan as const): kernels enqueued so far, optional per-step
  // event timing.  Calls on one plan are not thread-safe; give each host thread its own plan.
  mutable int64_t launches;
  mutable int prof_on, prof_n;
  mutable cudaEvent_t prof_ev[FBL_PROF_MAX + 1];
  mutable const char* prof_name[FBL_PROF_MAX];
};

static inline size_t fbl_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// Kernel launchers (all asynchronous on `st`; return a cudaError_t from the launch).
// ---------------------------------------------------------------------------------------------
struct GemmTerm {
  const void* a; int64_t a_rpad; int a_trans;   // logical A[m,k]; a_trans: stored as [k rows][m cols]
  const void* b; int64_t b_rpad; int b_trans;   // logical B[k,n]; b_trans: stored as [n rows][k cols]
  int k;
};
struct GemmArgs {
  int m, n, n_terms;
  GemmTerm t[4];
  void* c; int64_t c_rpad;        // C[m,n] stored [m rows][n cols]
  const float* bias;              // per output column, or nullptr
  const void* residual;           // same layout as C, or nullptr
  int seq, t_pad;                 // if t_pad > 0: rows with (row % t_pad) >= seq are written as zero
  int b_static;                   // 1: the first term's B operand is an input of the whole step (a weight)
  // optional fused row reduction D[b,h,t] = sum_d C[row, h*hd+d] * dot_with[row, h*hd+d] (fp32 C, before rounding)
  const void* dot_with; float* dot_out; int dot_hd, dot_hq;
  // reduction loop cut into ksplit slices whose fp32 partial tiles are added into `acc` (zeroed by the caller, same
  // element order as C with 4-byte elements); C itself is then produced from acc by launch_convert_f32_group
  int ksplit; float* acc;
  // of a group's first problem: chores of the launch (zero-fill zero_bytes, a multiple of 16, at zero_ptr for a
  // later kernel of the pass; reset the pass's status word), and `serial`: the launch may not start before
  // everything ahead of it on the stream has completed
  void* zero_ptr; size_t zero_bytes; int reset_status, serial;
  // fused activation of the feed-forward block (tensor-core kernel only): 0 none, 1 GELU forward (c = U, c2 = gelu(U)),
  // 2 GELU backward (c = value * gelu'(U), U in `residual`), 3 gated forward (c = G, c2 = silu(G) * U, U in `residual`),
  // 4 gated backward (c = value * silu(G), c2 = value * U * silu'(G); U in `residual`, G in `aux1`)
  int epi; const void* aux1; void* c2;
};

cudaError_t launch_gemm_simt(int dtype, const GemmArgs& g, cudaStream_t st);
bool gemm_tc_supported(const fbl_plan* p, const GemmArgs& g);
cudaError_t launch_gemm_tc_group(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st,
                                 int launch_id = -1);
struct GemmShape { int64_t m; int n; int kblocks; int splittable; };
int gemm_tc_choose_split(int sm_count, const GemmShape* sh, int count);
cudaError_t launch_wait_timeout_selftest(int32_t* status, long long limit_cycles, cudaStream_t st);
bool attn_fwd_tc_supported(const fbl_plan* p);
bool attn_bwd_tc_supported(const fbl_plan* p);
void fbl_note_cuda_error(cudaError_t e, const char* where);

cudaError_t launch_pack(int dtype, int unpack, const void* src, void* dst, int64_t outer, int64_t rows,
                        int64_t rows_pad, int cols, cudaStream_t st);
cudaError_t launch_rope(const fbl_plan* p, void* A, int heads_a, void* B, int heads_b, int inverse, cudaStream_t st);
bool norm_fwd_resets_status(const fbl_plan* p);   // the forward norm kernel for this plan zeroes the status word itself
cudaError_t launch_norm_fwd(const fbl_plan* p, const void* X, const float* gamma, const float* beta, void* Xn,
                            float* stats, int32_t* status, cudaStream_t st);
bool norm_bwd_takes_colsums(const fbl_plan* p);
cudaError_t launch_norm_bwd(const fbl_plan* p, const void* dXn, const void* X, const void* dY, const float* stats,
                            const float* gamma, void* dX, float* dgamma, float* dbeta, float* part,
                            cudaStream_t st, int bias_count = 0, const void* const* bias_m = nullptr,
                            const int* bias_cols = nullptr, float* const* bias_out = nullptr);
cudaError_t launch_colsum(int dtype, const void* M, int64_t rows, int64_t cols, float* out, float* partials,
                          cudaStream_t st);
size_t colsum_scratch_bytes(int64_t rows, int64_t cols);
cudaError_t launch_colsum_group(int dtype, int count, const void* const* M, int64_t rows, const int* cols,
                                float* const* out, float* partials, cudaStream_t st);

cudaError_t launch_attn_fwd_simt(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                                 cudaStream_t st);
cudaError_t launch_attn_bwd_simt(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* A,
                                 const void* dA, const float* lse, float* dvec, float* dqacc, void* dQ, void* dK,
                                 void* dV, cudaStream_t st);
cudaError_t launch_attn_bwd_pre(const fbl_plan* p, const void* A, const void* dA, float* dvec, float* dqacc,
                                bool dvec_ready, cudaStream_t st);
struct ConvertGroup { const float* src[4]; void* dst[4]; int64_t n[4]; int count; };
cudaError_t launch_convert_f32_group(const ConvertGroup& g, cudaStream_t st);   // bf16 destinations, n multiples of 4
cudaError_t launch_attn_bwd_post(const fbl_plan* p, const float* dqacc, void* dQ, cudaStream_t st);
cudaError_t launch_attn_fwd_tc(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                               int32_t* status, cudaStream_t st);
cudaError_t launch_attn_bwd_tc(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* A,
                               const void* dA, const float* lse, float* dvec, float* dqacc, void* dQ, void* dK,
                               void* dV, bool dvec_ready, int32_t* status, cudaStream_t st);
