// The attention layer with low-rank adapters on Q, K and V and frozen base weights: adapter storage, and the
// forward / backward drivers.  Every product runs on the layer's own GEMM kernels; the adapters' rank is padded
// to one 64-wide block each so that all operands are whole tiles.
#include <string.h>

#include "fbl_internal.h"

namespace {

constexpr int RB = FBL_LORA_BLOCK, RA = 3 * FBL_LORA_BLOCK;      // one adapter's block, all three

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & (FBL_ALIGN - 1)) != 0; }
inline int64_t up8(int64_t v) { return (v + 7) / 8 * 8; }

#define LORA_CUDA(expr)                                 \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) {                           \
      fbl_note_cuda_error(e__, #expr);                  \
      return FBL_ERR_CUDA;                              \
    }                                                   \
  } while (0)
#define LORA_STEP(name, kernels, expr)                                   \
  do {                                                                   \
    LORA_CUDA(expr);                                                     \
    p->launches += (kernels);                                            \
    if (p->prof_on && p->prof_n < FBL_PROF_MAX) {                        \
      p->prof_name[p->prof_n] = (name);                                  \
      LORA_CUDA(cudaEventRecord(p->prof_ev[1 + p->prof_n], st));         \
      p->prof_n++;                                                       \
    }                                                                    \
  } while (0)

// rows x cols block of a row-major matrix <-> the same block at (row_off, col_off) of an R-Tile matrix of r_pad rows
template <typename T>
__global__ void block_copy_kernel(const T* __restrict__ src, T* __restrict__ dst, int rows, int cols, int64_t r_pad,
                                  int row_off, int col_off, int unpack) {
  constexpr int TW = tile_w_of<T>::value;
  const int64_t total = (int64_t)rows * cols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / cols), c = (int)(i % cols);
    const int64_t t = rt_off<TW>(r_pad, row_off + r, col_off + c);
    if (unpack) dst[i] = src[t]; else dst[t] = src[i];
  }
}

// geometry of adapter `which`: block of A_all [d_model, 192] or of B_all [192, dq + 2 dkv]
bool adapter_block(const fbl_plan* p, int which, int* rows, int* cols, int64_t* r_pad, int* row_off, int* col_off) {
  const int D = p->d.d_model, r = p->lora_rank;
  const int colsB[3] = {p->dq, p->dkv, p->dkv}, offB[3] = {0, p->dq, p->dq + p->dkv};
  if (which >= FBL_LORA_AQ && which <= FBL_LORA_AV) {
    *rows = D; *cols = r; *r_pad = up8(D); *row_off = 0; *col_off = RB * (which - FBL_LORA_AQ);
    return true;
  }
  if (which >= FBL_LORA_BQ && which <= FBL_LORA_BV) {
    const int i = which - FBL_LORA_BQ;
    *rows = r; *cols = colsB[i]; *r_pad = RA; *row_off = RB * i; *col_off = offB[i];
    return true;
  }
  return false;
}

int pack_common(const fbl_plan* p, int which, const void* src, void* dst, void* stream, int unpack) {
  if (!p || !src || !dst || p->lora_rank <= 0) return FBL_ERR_INVALID_ARG;
  int rows, cols, row_off, col_off; int64_t r_pad;
  if (!adapter_block(p, which, &rows, &cols, &r_pad, &row_off, &col_off)) return FBL_ERR_INVALID_ARG;
  if (misaligned(unpack ? src : dst)) return FBL_ERR_MISALIGNED;
  const int blocks = (int)((int64_t)rows * cols / 256 + 1);
  if (p->d.dtype == FBL_DTYPE_FP32)
    block_copy_kernel<float><<<blocks, 256, 0, as_stream(stream)>>>((const float*)src, (float*)dst, rows, cols, r_pad, row_off, col_off, unpack);
  else
    block_copy_kernel<__nv_bfloat16><<<blocks, 256, 0, as_stream(stream)>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, cols, r_pad, row_off, col_off, unpack);
  LORA_CUDA(cudaGetLastError());
  return FBL_OK;
}

// column block `i` (q, k, v) of an R-Tile matrix with r_pad rows whose column blocks are dq, dkv, dkv wide
inline const char* colblock(const fbl_plan* p, const void* base, int64_t r_pad, int i) {
  const int off[3] = {0, p->dq, p->dq + p->dkv};
  return (const char*)base + (size_t)off[i] * (size_t)r_pad * p->e;     // whole 64 (32) column panels: panel stride r_pad * tw
}

cudaError_t run_group(const fbl_plan* p, GemmArgs* gs, int count, int32_t* status, cudaStream_t st, int* kernels) {
  bool tc = p->use_tc != 0;
  for (int i = 0; i < count; ++i) tc = tc && gemm_tc_supported(p, gs[i]);
  if (tc) { *kernels = 1; return launch_gemm_tc_group(p, gs, count, status, st); }
  *kernels = count;
  for (int i = 0; i < count; ++i) {
    cudaError_t e = launch_gemm_simt(p->d.dtype, gs[i], st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace

extern "C" {

int fbl_plan_enable_lora(fbl_plan* plan, int rank) {
  if (!plan || plan->cross || rank < 1 || rank > RB) return FBL_ERR_INVALID_ARG;
  if (plan->lora_rank > 0) return plan->lora_rank == rank ? FBL_OK : FBL_ERR_INVALID_ARG;
  plan->lora_rank = rank;
  const size_t n = (size_t)plan->n_pad;
  const size_t t_bytes = fbl_align_up(n * RA * (size_t)plan->e, FBL_ALIGN);
  plan->sv_t = plan->saved_bytes; plan->saved_bytes += t_bytes;
  plan->sb_dt = plan->scratch_bwd_bytes; plan->scratch_bwd_bytes += t_bytes;
  plan->sb_frozen = plan->scratch_bwd_bytes; plan->scratch_bwd_bytes += fbl_align_up(2 * (size_t)plan->d.d_model * sizeof(float), FBL_ALIGN);
  return FBL_OK;
}

int fbl_lora_bytes(const fbl_plan* plan, size_t* a_all_bytes, size_t* b_all_bytes) {
  if (!plan || plan->lora_rank <= 0) return FBL_ERR_INVALID_ARG;
  if (a_all_bytes) *a_all_bytes = (size_t)up8(plan->d.d_model) * RA * plan->e;
  if (b_all_bytes) *b_all_bytes = (size_t)RA * (plan->dq + 2 * plan->dkv) * plan->e;
  return FBL_OK;
}

int fbl_lora_pack(const fbl_plan* plan, int which, const void* rowmajor_dev, void* all_dev, void* stream) {
  return pack_common(plan, which, rowmajor_dev, all_dev, stream, 0);
}
int fbl_lora_unpack(const fbl_plan* plan, int which, const void* all_dev, void* rowmajor_dev, void* stream) {
  return pack_common(plan, which, all_dev, rowmajor_dev, stream, 1);
}

int fbl_layer_fwd_lora(const fbl_plan* p, const void* X, const float* gamma, const float* beta, const void* Wq,
                       const void* Wk, const void* Wv, const void* Wo, const float* bq, const float* bk, const float* bv,
                       const float* bo, const void* A_all, const void* B_all, void* Y, void* saved, void* scratch,
                       void* stream) {
  if (!p || p->lora_rank <= 0 || !X || !gamma || !Wq || !Wk || !Wv || !Wo || !A_all || !B_all || !Y || !saved || !scratch)
    return FBL_ERR_INVALID_ARG;
  if (p->d.has_bias && (!bq || !bk || !bv || !bo)) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !beta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {X, Wq, Wk, Wv, Wo, A_all, B_all, Y, saved, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  char* sv = (char*)saved;
  int32_t* status = (int32_t*)scratch;
  float* stats = (float*)(sv + p->sv_stats);
  void* Xn = sv + p->sv_xn; void* Q = sv + p->sv_q; void* K = sv + p->sv_k; void* V = sv + p->sv_v;
  void* A = sv + p->sv_a; float* lse = (float*)(sv + p->sv_lse); void* T = sv + p->sv_t;
  const bool bias = p->d.has_bias;
  const int n = (int)p->n_pad, D = p->d.d_model;
  int k = 0;

  if (!norm_fwd_resets_status(p)) LORA_CUDA(cudaMemsetAsync(status, 0, FBL_ALIGN, st));
  if (p->prof_on) { p->prof_n = 0; LORA_CUDA(cudaEventRecord(p->prof_ev[0], st)); }
  LORA_STEP("norm_fwd", 1, launch_norm_fwd(p, X, gamma, beta, Xn, stats, status, st));
  {
    GemmArgs g = {};                       // T = Xn [Aq | Ak | Av]: one thin product for the three adapters
    g.m = n; g.n = RA; g.n_terms = 1;
    g.t[0] = {Xn, p->n_pad, 0, A_all, up8(D), 0, D};
    g.b_static = 1;
    g.c = T; g.c_rpad = p->n_pad; g.seq = p->d.seq; g.t_pad = p->t_pad;
    LORA_CUDA(run_group(p, &g, 1, status, st, &k));
    LORA_STEP("lora_T", 0, cudaSuccess);
    p->launches += k;
  }
  {
    const void* W[3] = {Wq, Wk, Wv};
    void* O[3] = {Q, K, V};
    const float* B[3] = {bq, bk, bv};
    const int cols[3] = {p->dq, p->dkv, p->dkv};
    GemmArgs gs[3];
    for (int i = 0; i < 3; ++i) {         // Q = Xn Wq + T B_all[:, q block]: the rank is a second reduction loop
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = n; g.n = cols[i]; g.n_terms = 2;
      g.t[0] = {Xn, p->n_pad, 0, W[i], up8(D), 0, D};
      g.t[1] = {T, p->n_pad, 0, colblock(p, B_all, RA, i), RA, 0, RA};
      g.b_static = 1;
      g.c = O[i]; g.c_rpad = p->n_pad; g.bias = bias ? B[i] : nullptr;
      g.seq = p->d.seq; g.t_pad = p->t_pad;
    }
    LORA_CUDA(run_group(p, gs, 3, status, st, &k));
    LORA_STEP("proj_qkv", 0, cudaSuccess);
    p->launches += k;
  }
  if (p->rope_base > 0.f) LORA_STEP("rope", 1, launch_rope(p, Q, p->d.n_q_heads, K, p->d.n_kv_heads, 0, st));
  if (p->use_tc && attn_fwd_tc_supported(p)) LORA_STEP("attn_fwd", 1, launch_attn_fwd_tc(p, Q, K, V, A, lse, status, st));
  else LORA_STEP("attn_fwd", 1, launch_attn_fwd_simt(p, Q, K, V, A, lse, st));
  {
    GemmArgs g = {};
    g.m = n; g.n = D; g.n_terms = 1;
    g.t[0] = {A, p->n_pad, 0, Wo, up8(p->dq), 0, p->dq};
    g.b_static = 1;
    g.c = Y; g.c_rpad = p->n_pad; g.bias = bias ? bo : nullptr;
    g.residual = p->d.residual ? X : nullptr;
    g.seq = p->d.seq; g.t_pad = p->t_pad;
    LORA_CUDA(run_group(p, &g, 1, status, st, &k));
    LORA_STEP("proj_o", 0, cudaSuccess);
    p->launches += k;
  }
  return FBL_OK;
}

int fbl_layer_bwd_lora(const fbl_plan* p, const void* dY, const void* X, const float* gamma, const void* Wq,
                       const void* Wk, const void* Wv, const void* Wo, const void* A_all, const void* B_all,
                       const void* saved, void* dX, void* dA_all, void* dB_all, float* dgamma, float* dbeta,
                       void* scratch, void* stream) {
  if (!p || p->lora_rank <= 0 || !dY || !X || !gamma || !Wq || !Wk || !Wv || !Wo || !A_all || !B_all || !saved || !dX ||
      !dA_all || !dB_all || !scratch)
    return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {dY, X, Wq, Wk, Wv, Wo, A_all, B_all, saved, dX, dA_all, dB_all, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  const char* sv = (const char*)saved;
  char* sc = (char*)scratch;
  int32_t* status = (int32_t*)sc;
  const float* stats = (const float*)(sv + p->sv_stats);
  const void* Xn = sv + p->sv_xn; const void* Q = sv + p->sv_q; const void* K = sv + p->sv_k;
  const void* V = sv + p->sv_v; const void* A = sv + p->sv_a; const float* lse = (const float*)(sv + p->sv_lse);
  const void* T = sv + p->sv_t;
  void* dA = sc + p->sb_da; float* dvec = (float*)(sc + p->sb_dvec); float* dqacc = (float*)(sc + p->sb_dqacc);
  void* dQ = sc + p->sb_dq; void* dK = sc + p->sb_dk; void* dV = sc + p->sb_dv; void* dXn = sc + p->sb_dxn;
  void* dT = sc + p->sb_dt; float* part = (float*)(sc + p->sb_part);
  float* frozen = (float*)(sc + p->sb_frozen);                 // where the unused gradients of a frozen norm go
  if (!dgamma) dgamma = frozen;
  if (!dbeta) dbeta = frozen + p->d.d_model;
  const int n = (int)p->n_pad, D = p->d.d_model;
  const int cols[3] = {p->dq, p->dkv, p->dkv};
  int k = 0;

  LORA_CUDA(cudaMemsetAsync(status, 0, p->zero_bytes, st));    // status word and the dQ accumulator
  if (p->prof_on) { p->prof_n = 0; LORA_CUDA(cudaEventRecord(p->prof_ev[0], st)); }
  bool dvec_ready = false;
  {
    GemmArgs ga = {};                      // dA = dY Wo^T; dWo is not formed: Wo is frozen
    ga.m = n; ga.n = p->dq; ga.n_terms = 1;
    ga.t[0] = {dY, p->n_pad, 0, Wo, up8(p->dq), 1, D};
    ga.b_static = 1;
    ga.c = dA; ga.c_rpad = p->n_pad; ga.seq = p->d.seq; ga.t_pad = p->t_pad;
    if (p->use_tc && gemm_tc_supported(p, ga)) {
      ga.dot_with = A; ga.dot_out = dvec; ga.dot_hd = p->d.head_dim; ga.dot_hq = p->d.n_q_heads;
      dvec_ready = true;
    }
    LORA_CUDA(run_group(p, &ga, 1, status, st, &k));
    LORA_STEP("dA", 0, cudaSuccess);
    p->launches += k;
  }
  if (p->use_tc && attn_bwd_tc_supported(p)) LORA_STEP("attn_bwd", dvec_ready ? 2 : 3, launch_attn_bwd_tc(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, dvec_ready, status, st));
  else LORA_STEP("attn_bwd", 3, launch_attn_bwd_simt(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, st));
  if (p->rope_base > 0.f) LORA_STEP("rope_bwd", 1, launch_rope(p, dQ, p->d.n_q_heads, dK, p->d.n_kv_heads, 1, st));
  const void* G[3] = {dQ, dK, dV};
  {
    GemmArgs g = {};                       // dT = dQ Bq^T | dK Bk^T | dV Bv^T: B_all's column blocks read with swapped axes;
    g.m = n; g.n = RA; g.n_terms = 3;      // its zero blocks keep each gradient in its own adapter's columns
    for (int i = 0; i < 3; ++i) g.t[i] = {G[i], p->n_pad, 0, colblock(p, B_all, RA, i), RA, 1, cols[i]};
    g.c = dT; g.c_rpad = p->n_pad; g.seq = p->d.seq; g.t_pad = p->t_pad;
    LORA_CUDA(run_group(p, &g, 1, status, st, &k));
    LORA_STEP("lora_dT", 0, cudaSuccess);
    p->launches += k;
  }
  {
    GemmArgs gs[5];
    for (int i = 0; i < 3; ++i) {          // dB_all[:, block i] = T^T d*: token-axis reduction, T's tiles read MN-major
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = RA; g.n = cols[i]; g.n_terms = 1;
      g.t[0] = {T, p->n_pad, 1, G[i], p->n_pad, 0, n};
      g.c = (void*)colblock(p, dB_all, RA, i); g.c_rpad = RA;
    }
    GemmArgs& gx = gs[3];                  // dXn = dQ Wq^T + dK Wk^T + dV Wv^T + dT A_all^T: four reduction loops
    gx = GemmArgs{};
    gx.m = n; gx.n = D; gx.n_terms = 4;
    const void* W[3] = {Wq, Wk, Wv};
    for (int i = 0; i < 3; ++i) gx.t[i] = {G[i], p->n_pad, 0, W[i], up8(D), 1, cols[i]};
    gx.t[3] = {dT, p->n_pad, 0, A_all, up8(D), 1, RA};
    gx.b_static = 0;
    gx.c = dXn; gx.c_rpad = p->n_pad; gx.seq = p->d.seq; gx.t_pad = p->t_pad;
    GemmArgs& g = gs[4];                   // dA_all = Xn^T dT: token-axis reduction, in the same launch
    g = GemmArgs{};
    g.m = D; g.n = RA; g.n_terms = 1;
    g.t[0] = {Xn, p->n_pad, 1, dT, p->n_pad, 0, n};
    g.c = dA_all; g.c_rpad = up8(D);
    LORA_CUDA(run_group(p, gs, 5, status, st, &k));
    LORA_STEP("dB+dXn+dA", 0, cudaSuccess);
    p->launches += k;
  }
  LORA_STEP("norm_bwd", norm_bwd_takes_colsums(p) ? 2 : 1, launch_norm_bwd(p, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, part, st));
  return FBL_OK;
}

}  // extern "C"
