// Cross-attention layer: forward and backward drivers.  K and V come from a memory sequence with its own length and
// width; every kernel is the self-attention layer's (the attention kernels take the key side's geometry from the
// plan), so the second sequence needs no transposition or re-partitioning either.
#include <string.h>

#include "fbl_internal.h"

namespace {

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & (FBL_ALIGN - 1)) != 0; }
inline int64_t up8(int64_t v) { return (v + 7) / 8 * 8; }

#define XA_CUDA(expr)                                   \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) {                           \
      fbl_note_cuda_error(e__, #expr);                  \
      return FBL_ERR_CUDA;                              \
    }                                                   \
  } while (0)
#define XA_STEP(name, kernels, expr)                                     \
  do {                                                                   \
    XA_CUDA(expr);                                                       \
    p->launches += (kernels);                                            \
    if (p->prof_on && p->prof_n < FBL_PROF_MAX) {                        \
      p->prof_name[p->prof_n] = (name);                                  \
      XA_CUDA(cudaEventRecord(p->prof_ev[1 + p->prof_n], st));           \
      p->prof_n++;                                                       \
    }                                                                    \
  } while (0)
#define XA_PROF_BEGIN() \
  do { if (p->prof_on) { p->prof_n = 0; XA_CUDA(cudaEventRecord(p->prof_ev[0], st)); } } while (0)

cudaError_t run_gemm(const fbl_plan* p, const GemmArgs& g, int32_t* status, cudaStream_t st) {
  if (p->use_tc && gemm_tc_supported(p, g)) return launch_gemm_tc_group(p, &g, 1, status, st);
  return launch_gemm_simt(p->d.dtype, g, st);
}

}  // namespace

extern "C" {

int fbl_xattn_fwd(const fbl_plan* p, const void* X, const void* M, const float* gamma, const float* beta, const void* Wq,
                  const void* Wk, const void* Wv, const void* Wo, const float* bq, const float* bk, const float* bv,
                  const float* bo, void* Y, void* saved, void* scratch, void* stream) {
  if (!p || !X || !M || !gamma || !Wq || !Wk || !Wv || !Wo || !Y || !saved || !scratch) return FBL_ERR_INVALID_ARG;
  if (!p->cross) return FBL_ERR_INVALID_ARG;
  if (p->d.has_bias && (!bq || !bk || !bv || !bo)) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !beta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {X, M, Wq, Wk, Wv, Wo, Y, saved, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  char* sv = (char*)saved;
  int32_t* status = (int32_t*)scratch;
  float* stats = (float*)(sv + p->sv_stats);
  void* Xn = sv + p->sv_xn; void* Q = sv + p->sv_q; void* K = sv + p->sv_k; void* V = sv + p->sv_v;
  void* A = sv + p->sv_a; float* lse = (float*)(sv + p->sv_lse);
  const bool bias = p->d.has_bias;
  const int n = (int)p->n_pad, nk = (int)p->n_pad_kv, D = p->d.d_model, Dm = p->d_mem;

  if (!norm_fwd_resets_status(p)) XA_CUDA(cudaMemsetAsync(status, 0, FBL_ALIGN, st));
  XA_PROF_BEGIN();
  XA_STEP("norm_fwd", 1, launch_norm_fwd(p, X, gamma, beta, Xn, stats, status, st));
  {
    // Q from the normalised hidden states, K and V from the memory: three problems with their own row counts and
    // reduction lengths, one launch
    GemmArgs gs[3];
    for (int i = 0; i < 3; ++i) gs[i] = GemmArgs{};
    gs[0].m = n; gs[0].n = p->dq; gs[0].n_terms = 1;
    gs[0].t[0] = {Xn, p->n_pad, 0, Wq, D, 0, D};
    gs[0].c = Q; gs[0].c_rpad = p->n_pad; gs[0].bias = bias ? bq : nullptr; gs[0].seq = p->d.seq; gs[0].t_pad = p->t_pad;
    const void* W[2] = {Wk, Wv};
    void* O[2] = {K, V};
    const float* B[2] = {bk, bv};
    for (int i = 0; i < 2; ++i) {
      GemmArgs& g = gs[1 + i];
      g.m = nk; g.n = p->dkv; g.n_terms = 1;
      g.t[0] = {M, p->n_pad_kv, 0, W[i], up8(Dm), 0, Dm};
      g.c = O[i]; g.c_rpad = p->n_pad_kv; g.bias = bias ? B[i] : nullptr; g.seq = p->seq_kv; g.t_pad = p->t_pad_kv;
    }
    bool tc = p->use_tc != 0;
    for (int i = 0; i < 3; ++i) { gs[i].b_static = 1; tc = tc && gemm_tc_supported(p, gs[i]); }
    if (tc) {
      XA_STEP("proj_qkv", 1, launch_gemm_tc_group(p, gs, 3, status, st));
    } else {
      for (int i = 0; i < 3; ++i)
        XA_STEP(i == 0 ? "proj_q" : i == 1 ? "proj_k" : "proj_v", 1, run_gemm(p, gs[i], status, st));
    }
  }
  if (p->use_tc && attn_fwd_tc_supported(p)) XA_STEP("attn_fwd", 1, launch_attn_fwd_tc(p, Q, K, V, A, lse, status, st));
  else XA_STEP("attn_fwd", 1, launch_attn_fwd_simt(p, Q, K, V, A, lse, st));
  {
    GemmArgs g = {};
    g.m = n; g.n = D; g.n_terms = 1;
    g.t[0] = {A, p->n_pad, 0, Wo, up8(p->dq), 0, p->dq};
    g.b_static = 1;
    g.c = Y; g.c_rpad = p->n_pad; g.bias = bias ? bo : nullptr;
    g.residual = p->d.residual ? X : nullptr;
    g.seq = p->d.seq; g.t_pad = p->t_pad;
    XA_STEP("proj_o", 1, run_gemm(p, g, status, st));
  }
  return FBL_OK;
}

int fbl_xattn_bwd(const fbl_plan* p, const void* dY, const void* X, const void* M, const float* gamma, const void* Wq,
                  const void* Wk, const void* Wv, const void* Wo, const void* saved, void* dX, void* dM, void* dWq,
                  void* dWk, void* dWv, void* dWo, float* dbq, float* dbk, float* dbv, float* dbo, float* dgamma,
                  float* dbeta, void* scratch, void* stream) {
  if (!p || !dY || !X || !M || !gamma || !Wq || !Wk || !Wv || !Wo || !saved || !dX || !dM || !dWq || !dWk || !dWv ||
      !dWo || !dgamma || !scratch)
    return FBL_ERR_INVALID_ARG;
  if (!p->cross) return FBL_ERR_INVALID_ARG;
  if (p->d.has_bias && (!dbq || !dbk || !dbv || !dbo)) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !dbeta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {dY, X, M, Wq, Wk, Wv, Wo, saved, dX, dM, dWq, dWk, dWv, dWo, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  const char* sv = (const char*)saved;
  char* sc = (char*)scratch;
  int32_t* status = (int32_t*)sc;
  const float* stats = (const float*)(sv + p->sv_stats);
  const void* Xn = sv + p->sv_xn; const void* Q = sv + p->sv_q; const void* K = sv + p->sv_k;
  const void* V = sv + p->sv_v; const void* A = sv + p->sv_a; const float* lse = (const float*)(sv + p->sv_lse);
  void* dA = sc + p->sb_da; float* dvec = (float*)(sc + p->sb_dvec); float* dqacc = (float*)(sc + p->sb_dqacc);
  void* dQ = sc + p->sb_dq; void* dK = sc + p->sb_dk; void* dV = sc + p->sb_dv; void* dXn = sc + p->sb_dxn;
  float* part = (float*)(sc + p->sb_part);
  float* part_kv = (float*)(sc + p->sb_part_kv);
  const bool bias = p->d.has_bias;
  const int n = (int)p->n_pad, nk = (int)p->n_pad_kv, D = p->d.d_model, Dm = p->d_mem;

  // one fill: status word, the accumulation areas of sliced weight-gradient products, the dQ accumulator.  It is
  // also the barrier between the forward pass's kernels and the backward's, which the attention backward relies on
  // when it requests forward-pass data before waiting for the kernel in front of it.
  XA_CUDA(cudaMemsetAsync(status, 0, p->zero_bytes, st));
  XA_PROF_BEGIN();
  const bool split_o = p->use_tc && p->ksplit_o > 1, split_q = p->use_tc && p->ksplit_qkv > 1,
             split_kv = p->use_tc && p->ksplit_kv > 1;
  ConvertGroup cg = {};                     // sliced products leave fp32 sums; one launch rounds them all at the end
  bool dvec_ready = false;
  {
    GemmArgs gs[2];
    GemmArgs& gw = gs[0];                   // dWo = A^T dY
    gw = GemmArgs{};
    gw.m = p->dq; gw.n = D; gw.n_terms = 1;
    gw.t[0] = {A, p->n_pad, 1, dY, p->n_pad, 0, n};
    gw.c = dWo; gw.c_rpad = up8(p->dq);
    GemmArgs& ga = gs[1];                   // dA = dY Wo^T
    ga = GemmArgs{};
    ga.m = n; ga.n = p->dq; ga.n_terms = 1;
    ga.t[0] = {dY, p->n_pad, 0, Wo, up8(p->dq), 1, D};
    ga.b_static = 1;
    ga.c = dA; ga.c_rpad = p->n_pad; ga.seq = p->d.seq; ga.t_pad = p->t_pad;
    if (p->use_tc && gemm_tc_supported(p, gw) && gemm_tc_supported(p, ga)) {
      ga.dot_with = A; ga.dot_out = dvec; ga.dot_hd = p->d.head_dim; ga.dot_hq = p->d.n_q_heads;
      dvec_ready = true;
      if (split_o) {
        gw.ksplit = p->ksplit_o; gw.acc = (float*)(sc + p->sb_acc_o);
        cg.src[cg.count] = gw.acc; cg.dst[cg.count] = dWo; cg.n[cg.count] = up8(p->dq) * (int64_t)D; cg.count++;
      }
      XA_STEP("dWo+dA", 1, launch_gemm_tc_group(p, gs, 2, status, st));
    } else {
      XA_STEP("dA", 1, run_gemm(p, ga, status, st));
      XA_STEP("dWo", 1, run_gemm(p, gw, status, st));
    }
  }
  if (p->use_tc && attn_bwd_tc_supported(p)) XA_STEP("attn_bwd", dvec_ready ? 2 : 3, launch_attn_bwd_tc(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, dvec_ready, status, st));
  else XA_STEP("attn_bwd", 3, launch_attn_bwd_simt(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, st));
  {
    // query side: dWq = Xn^T dQ (token-axis reduction), dXn = dQ Wq^T
    // memory side: dWk = M^T dK, dWv = M^T dV (reductions over the memory's tokens), dM = dK Wk^T + dV Wv^T
    GemmArgs gq[2], gk[3];
    gq[0] = GemmArgs{};
    gq[0].m = D; gq[0].n = p->dq; gq[0].n_terms = 1;
    gq[0].t[0] = {Xn, p->n_pad, 1, dQ, p->n_pad, 0, n};
    gq[0].c = dWq; gq[0].c_rpad = up8(D);
    gq[1] = GemmArgs{};
    gq[1].m = n; gq[1].n = D; gq[1].n_terms = 1;
    gq[1].t[0] = {dQ, p->n_pad, 0, Wq, up8(D), 1, p->dq};
    gq[1].b_static = 1;
    gq[1].c = dXn; gq[1].c_rpad = p->n_pad; gq[1].seq = p->d.seq; gq[1].t_pad = p->t_pad;
    const void* G[2] = {dK, dV};
    void* DW[2] = {dWk, dWv};
    for (int i = 0; i < 2; ++i) {
      gk[i] = GemmArgs{};
      gk[i].m = Dm; gk[i].n = p->dkv; gk[i].n_terms = 1;
      gk[i].t[0] = {M, p->n_pad_kv, 1, G[i], p->n_pad_kv, 0, nk};
      gk[i].c = DW[i]; gk[i].c_rpad = up8(Dm);
    }
    gk[2] = GemmArgs{};
    gk[2].m = nk; gk[2].n = Dm; gk[2].n_terms = 2;
    gk[2].t[0] = {dK, p->n_pad_kv, 0, Wk, up8(Dm), 1, p->dkv};
    gk[2].b_static = 1;
    gk[2].t[1] = {dV, p->n_pad_kv, 0, Wv, up8(Dm), 1, p->dkv};
    gk[2].c = dM; gk[2].c_rpad = p->n_pad_kv; gk[2].seq = p->seq_kv; gk[2].t_pad = p->t_pad_kv;
    bool tc_q = p->use_tc != 0, tc_k = p->use_tc != 0;
    for (int i = 0; i < 2; ++i) tc_q = tc_q && gemm_tc_supported(p, gq[i]);
    for (int i = 0; i < 3; ++i) tc_k = tc_k && gemm_tc_supported(p, gk[i]);
    if (tc_q && split_q) {
      gq[0].ksplit = p->ksplit_qkv; gq[0].acc = (float*)(sc + p->sb_acc_qkv);
      cg.src[cg.count] = gq[0].acc; cg.dst[cg.count] = dWq; cg.n[cg.count] = up8(D) * (int64_t)p->dq; cg.count++;
    }
    if (tc_k && split_kv) {
      float* acc = (float*)(sc + p->sb_acc_kv);
      for (int i = 0; i < 2; ++i) {
        gk[i].ksplit = p->ksplit_kv; gk[i].acc = acc;
        cg.src[cg.count] = acc; cg.dst[cg.count] = DW[i]; cg.n[cg.count] = up8(Dm) * (int64_t)p->dkv; cg.count++;
        acc += up8(Dm) * (int64_t)p->dkv;
      }
    }
    if (tc_q && tc_k) {
      // both sides in one launch: the three token-axis reductions first in the work list (longest loops), then the
      // two input gradients
      GemmArgs all[5] = {gq[0], gk[0], gk[1], gq[1], gk[2]};
      XA_STEP("dWqkv+dXn+dM", 1, launch_gemm_tc_group(p, all, 5, status, st));
    } else {
    if (tc_q) {
      XA_STEP("dWq+dXn", 1, launch_gemm_tc_group(p, gq, 2, status, st));
    } else {
      XA_STEP("dXn", 1, run_gemm(p, gq[1], status, st));
      XA_STEP("dWq", 1, run_gemm(p, gq[0], status, st));
    }
    if (tc_k) {
      XA_STEP("dWkv+dM", 1, launch_gemm_tc_group(p, gk, 3, status, st));
    } else {
      XA_STEP("dM", 1, run_gemm(p, gk[2], status, st));
      XA_STEP("dWk", 1, run_gemm(p, gk[0], status, st));
      XA_STEP("dWv", 1, run_gemm(p, gk[1], status, st));
    }
    }
    if (cg.count > 0) XA_STEP("dW round", 1, launch_convert_f32_group(cg, st));
  }
  // bias gradients: column sums over the query tokens (dY, dQ) and over the memory's tokens (dK, dV)
  const void* Mq[2] = {dY, dQ};
  float* Oq[2] = {dbo, dbq};
  const int Cq[2] = {D, p->dq};
  const void* Mk[2] = {dK, dV};
  float* Ok[2] = {dbk, dbv};
  const int Ck[2] = {p->dkv, p->dkv};
  if (bias) XA_STEP("db_kv", 2, launch_colsum_group(p->d.dtype, 2, Mk, p->n_pad_kv, Ck, Ok, part_kv, st));
  if (bias && norm_bwd_takes_colsums(p)) {
    XA_STEP("db+norm_bwd", 2, launch_norm_bwd(p, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, part, st, 2, Mq, Cq, Oq));
    return FBL_OK;
  }
  if (bias) XA_STEP("db", 2, launch_colsum_group(p->d.dtype, 2, Mq, p->n_pad, Cq, Oq, part, st));
  XA_STEP("norm_bwd", norm_bwd_takes_colsums(p) ? 2 : 1, launch_norm_bwd(p, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, part, st));
  return FBL_OK;
}

}  // extern "C"
