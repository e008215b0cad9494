// The feed-forward half of the block: plan, work-area layout, activation kernels and the forward/backward drivers.
// Its six (nine, gated) matmuls run on the same GEMM kernels as the attention layer's projections, with the same
// operand-orientation flags instead of transposes; the norm and the bias column sums are the attention layer's too.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "fbl_internal.h"
#include "pdl.cuh"

struct fbl_mlp_plan {
  fbl_mlp_desc d;
  fbl_plan* base;            // carries what the shared launchers read: dtype, token geometry, d_model, norm, SM count, knobs
  int64_t n_pad;
  size_t sv_stats, sv_xn, sv_u, sv_g, sv_h, saved_bytes;
  size_t sb_acc2, sb_acc1, zero_bytes, sb_dh, sb_du, sb_dg, sb_dxn, sb_part, part_bytes, scratch_bwd_bytes, scratch_fwd_bytes;
  int ksplit_2, ksplit_1;    // reduction slices of dW2 and of dW1 / dWg (1: none)
  mutable int64_t launches;
};

namespace {

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & (FBL_ALIGN - 1)) != 0; }
inline int64_t up8(int64_t v) { return (v + 7) / 8 * 8; }

#define MLP_CUDA(expr)                                  \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) {                           \
      fbl_note_cuda_error(e__, #expr);                  \
      return FBL_ERR_CUDA;                              \
    }                                                   \
  } while (0)
#define MLP_STEP(kernels, expr) do { MLP_CUDA(expr); p->launches += (kernels); } while (0)

constexpr float GELU_K0 = 0.7978845608028654f, GELU_K1 = 0.044715f;

__device__ __forceinline__ float gelu_f(float u) {
  return 0.5f * u * (1.f + tanhf(GELU_K0 * (u + GELU_K1 * u * u * u)));
}
__device__ __forceinline__ float gelu_grad_f(float u) {
  const float t = tanhf(GELU_K0 * (u + GELU_K1 * u * u * u));
  return 0.5f * (1.f + t) + 0.5f * u * (1.f - t * t) * GELU_K0 * (1.f + 3.f * GELU_K1 * u * u);
}
__device__ __forceinline__ float sigmoid_f(float g) { return 1.f / (1.f + __expf(-g)); }

template <typename T> struct V16 { static constexpr int N = 16 / (int)sizeof(T); };

template <typename T>
__device__ __forceinline__ void ld16(const T* p, float (&v)[V16<T>::N]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < V16<T>::N; ++i) v[i] = to_f(e[i]);
}
template <typename T>
__device__ __forceinline__ void st16(T* p, const float (&v)[V16<T>::N]) {
  uint4 raw;
  T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
  for (int i = 0; i < V16<T>::N; ++i) e[i] = from_f<T>(v[i]);
  *reinterpret_cast<uint4*>(p) = raw;
}

// H = gelu(U) or silu(G) * U over whole padded buffers (all three share one shape and tile order, so the pass is
// flat; padding slots hold zeros and map to zero).  16-byte accesses, grid-stride.
template <typename T, bool GATED>
__global__ void __launch_bounds__(256) act_fwd_kernel(const T* __restrict__ U, const T* __restrict__ G, T* __restrict__ H,
                                                      int64_t n_vec) {
  constexpr int V = V16<T>::N;
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * blockDim.x) {
    float u[V], h[V];
    ld16(U + i * V, u);
    if (GATED) {
      float g[V];
      ld16(G + i * V, g);
#pragma unroll
      for (int k = 0; k < V; ++k) h[k] = g[k] * sigmoid_f(g[k]) * u[k];
    } else {
#pragma unroll
      for (int k = 0; k < V; ++k) h[k] = gelu_f(u[k]);
    }
    st16(H + i * V, h);
  }
}

// dU = dH gelu'(U), or dU = dH silu(G) and dG = dH U silu'(G)
template <typename T, bool GATED>
__global__ void __launch_bounds__(256) act_bwd_kernel(const T* __restrict__ dH, const T* __restrict__ U,
                                                      const T* __restrict__ G, T* __restrict__ dU, T* __restrict__ dG,
                                                      int64_t n_vec) {
  constexpr int V = V16<T>::N;
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * blockDim.x) {
    float dh[V], u[V], du[V];
    ld16(dH + i * V, dh);
    ld16(U + i * V, u);
    if (GATED) {
      float g[V], dg[V];
      ld16(G + i * V, g);
#pragma unroll
      for (int k = 0; k < V; ++k) {
        const float s = sigmoid_f(g[k]);
        du[k] = dh[k] * g[k] * s;
        dg[k] = dh[k] * u[k] * s * (1.f + g[k] * (1.f - s));
      }
      st16(dG + i * V, dg);
    } else {
#pragma unroll
      for (int k = 0; k < V; ++k) du[k] = dh[k] * gelu_grad_f(u[k]);
    }
    st16(dU + i * V, du);
  }
}

template <typename T>
cudaError_t act_launch(const fbl_mlp_plan* p, bool bwd, const void* a, const void* U, const void* G, void* o1, void* o2,
                       cudaStream_t st) {
  const int64_t n_vec = p->n_pad * p->d.d_ff / V16<T>::N;
  const int blocks = (int)min((int64_t)p->base->sm_count * 8, (n_vec + 255) / 256);
  const bool gated = p->d.act == FBL_ACT_SWIGLU;
  if (!bwd) {
    if (gated) return launch_pdl(act_fwd_kernel<T, true>, dim3(blocks), dim3(256), 0, st, (const T*)U, (const T*)G, (T*)o1, n_vec);
    return launch_pdl(act_fwd_kernel<T, false>, dim3(blocks), dim3(256), 0, st, (const T*)U, (const T*)G, (T*)o1, n_vec);
  }
  if (gated) return launch_pdl(act_bwd_kernel<T, true>, dim3(blocks), dim3(256), 0, st, (const T*)a, (const T*)U, (const T*)G, (T*)o1, (T*)o2, n_vec);
  return launch_pdl(act_bwd_kernel<T, false>, dim3(blocks), dim3(256), 0, st, (const T*)a, (const T*)U, (const T*)G, (T*)o1, (T*)o2, n_vec);
}

cudaError_t act(const fbl_mlp_plan* p, bool bwd, const void* a, const void* U, const void* G, void* o1, void* o2, cudaStream_t st) {
  return p->d.dtype == FBL_DTYPE_FP32 ? act_launch<float>(p, bwd, a, U, G, o1, o2, st)
                                      : act_launch<__nv_bfloat16>(p, bwd, a, U, G, o1, o2, st);
}

// One launch for a group of problems on the tensor-core kernel if every one of them can run there, else one FFMA
// launch per problem.  Returns the number of kernels enqueued in *kernels.
cudaError_t run_group(const fbl_mlp_plan* p, GemmArgs* gs, int count, int32_t* status, cudaStream_t st, int* kernels) {
  bool tc = p->base->use_tc != 0;
  for (int i = 0; i < count; ++i) tc = tc && gemm_tc_supported(p->base, gs[i]);
  if (tc) { *kernels = 1; return launch_gemm_tc_group(p->base, gs, count, status, st); }
  *kernels = count;
  for (int i = 0; i < count; ++i) {
    gs[i].ksplit = 0; gs[i].acc = nullptr;
    cudaError_t e = launch_gemm_simt(p->d.dtype, gs[i], st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

bool mshape(const fbl_mlp_plan* p, int id, int64_t* outer, int64_t* rows, int64_t* rows_pad, int* cols) {
  const fbl_mlp_desc& d = p->d;
  switch (id) {
    case FBL_MT_X: *outer = d.batch; *rows = d.seq; *rows_pad = up8(d.seq); *cols = d.d_model; return true;
    case FBL_MT_H: *outer = d.batch; *rows = d.seq; *rows_pad = up8(d.seq); *cols = d.d_ff; return true;
    case FBL_MT_W1: *outer = 1; *rows = d.d_model; *rows_pad = up8(d.d_model); *cols = d.d_ff; return true;
    case FBL_MT_W2: *outer = 1; *rows = d.d_ff; *rows_pad = up8(d.d_ff); *cols = d.d_model; return true;
    default: return false;
  }
}

}  // namespace

extern "C" {

int fbl_mlp_plan_create(const fbl_mlp_desc* desc, fbl_mlp_plan** out) {
  if (!desc || !out) return FBL_ERR_INVALID_ARG;
  *out = nullptr;
  const fbl_mlp_desc& d = *desc;
  if (d.batch <= 0 || d.seq <= 0 || d.d_model <= 0 || d.d_ff <= 0) return FBL_ERR_INVALID_ARG;
  if (d.act != FBL_ACT_GELU && d.act != FBL_ACT_SWIGLU) return FBL_ERR_INVALID_ARG;
  const int e = d.dtype == FBL_DTYPE_FP32 ? 4 : 2, tw = 128 / e;
  if (d.d_model % tw != 0 || d.d_ff % tw != 0) return FBL_ERR_UNSUPPORTED_SHAPE;     // whole tiles (section 4.3)
  if (d.d_ff > (1 << 20)) return FBL_ERR_UNSUPPORTED_SHAPE;
  // the shared launchers read the token geometry, dtype, norm, SM count and knobs from an attention-layer plan of
  // the same batch, sequence and width (one head per tile column so that any d_model passes its checks)
  fbl_layer_desc ld = {};
  ld.batch = d.batch; ld.seq = d.seq; ld.d_model = d.d_model; ld.head_dim = d.dtype == FBL_DTYPE_FP32 ? 32 : 64;
  ld.n_q_heads = ld.n_kv_heads = 1; ld.dtype = d.dtype; ld.norm = d.norm; ld.causal = 0; ld.has_bias = d.has_bias;
  ld.residual = d.residual; ld.eps = d.eps; ld.softmax_scale = 0.f;
  fbl_plan* base = nullptr;
  int rc = fbl_plan_create(&ld, &base);
  if (rc != FBL_OK) return rc;
  fbl_mlp_plan* p = new (std::nothrow) fbl_mlp_plan();
  if (!p) { fbl_plan_destroy(base); return FBL_ERR_INVALID_ARG; }
  p->d = d; p->base = base; p->n_pad = base->n_pad; p->launches = 0;
  const size_t n = (size_t)p->n_pad;
  auto mat = [&](size_t cols) { return fbl_align_up(n * cols * (size_t)e, FBL_ALIGN); };
  const bool gated = d.act == FBL_ACT_SWIGLU;
  size_t o = 0;
  p->sv_stats = o; o += fbl_align_up(n * 2 * sizeof(float), FBL_ALIGN);
  p->sv_xn = o; o += mat(d.d_model);
  p->sv_u = o; o += mat(d.d_ff);
  p->sv_g = o; if (gated) o += mat(d.d_ff);
  p->sv_h = o; o += mat(d.d_ff);
  p->saved_bytes = o;
  p->scratch_fwd_bytes = FBL_ALIGN;

  // weight-gradient products reduce over all tokens: slice that reduction where it balances the SMs
  p->ksplit_2 = p->ksplit_1 = 1;
  if (base->use_tc) {
    const int kb_tok = (int)((p->n_pad + 63) / 64);
    const GemmShape g2[2] = {{d.d_ff, d.d_model, kb_tok, 1}, {p->n_pad, d.d_ff, (d.d_model + 63) / 64, 0}};
    p->ksplit_2 = gemm_tc_choose_split(base->sm_count, g2, 2);
    const GemmShape g1[3] = {{d.d_model, d.d_ff, kb_tok, 1}, {d.d_model, d.d_ff, kb_tok, 1},
                             {p->n_pad, d.d_model, (int)((gated ? 2 : 1) * ((d.d_ff + 63) / 64)), 0}};
    if (gated) p->ksplit_1 = gemm_tc_choose_split(base->sm_count, g1, 3);
    else { const GemmShape g1n[2] = {g1[0], g1[2]}; p->ksplit_1 = gemm_tc_choose_split(base->sm_count, g1n, 2); }
    if (getenv("FBL_KSPLIT_MLP")) p->ksplit_2 = p->ksplit_1 = atoi(getenv("FBL_KSPLIT_MLP"));     // tuning / test knob
  }
  o = FBL_ALIGN;   // status word, then the fp32 accumulation areas of sliced reductions (zero-filled together)
  p->sb_acc2 = o; if (p->ksplit_2 > 1) o += fbl_align_up((size_t)up8(d.d_ff) * d.d_model * sizeof(float), FBL_ALIGN);
  p->sb_acc1 = o; if (p->ksplit_1 > 1) o += fbl_align_up((size_t)up8(d.d_model) * d.d_ff * sizeof(float) * (gated ? 2 : 1), FBL_ALIGN);
  p->zero_bytes = o;
  p->sb_dh = o; o += mat(d.d_ff);
  p->sb_du = o; o += mat(d.d_ff);
  p->sb_dg = o; if (gated) o += mat(d.d_ff);
  p->sb_dxn = o; o += mat(d.d_model);
  {
    const size_t cs_floats = colsum_scratch_bytes(p->n_pad, (int64_t)d.d_model + 2 * (int64_t)d.d_ff) / sizeof(float);
    const size_t norm_floats = (size_t)2 * base->sm_count * 2 * d.d_model;
    p->part_bytes = fbl_align_up(((cs_floats + 255) / 256 * 256 + norm_floats) * sizeof(float), FBL_ALIGN);
  }
  p->sb_part = o; o += p->part_bytes;
  p->scratch_bwd_bytes = o;
  *out = p;
  return FBL_OK;
}

void fbl_mlp_plan_destroy(fbl_mlp_plan* plan) {
  if (!plan) return;
  fbl_plan_destroy(plan->base);
  delete plan;
}

int fbl_mlp_set_kernel_path(fbl_mlp_plan* plan, int path) {
  if (!plan) return FBL_ERR_INVALID_ARG;
  return fbl_plan_set_kernel_path(plan->base, path);
}
int64_t fbl_mlp_launch_count(const fbl_mlp_plan* plan) { return plan ? plan->launches : -1; }

int fbl_mlp_tensor_bytes(const fbl_mlp_plan* plan, int matrix_id, size_t* bytes) {
  int64_t outer, rows, rows_pad; int cols;
  if (!plan || !bytes || !mshape(plan, matrix_id, &outer, &rows, &rows_pad, &cols)) return FBL_ERR_INVALID_ARG;
  *bytes = (size_t)(outer * rows_pad) * cols * plan->base->e;
  return FBL_OK;
}

int fbl_mlp_workspace_bytes(const fbl_mlp_plan* plan, size_t* saved, size_t* scratch_fwd, size_t* scratch_bwd) {
  if (!plan) return FBL_ERR_INVALID_ARG;
  if (saved) *saved = plan->saved_bytes;
  if (scratch_fwd) *scratch_fwd = plan->scratch_fwd_bytes;
  if (scratch_bwd) *scratch_bwd = plan->scratch_bwd_bytes;
  return FBL_OK;
}

int fbl_mlp_workspace_offset(const fbl_mlp_plan* plan, int what, size_t* offset, size_t* bytes) {
  if (!plan || !offset || !bytes) return FBL_ERR_INVALID_ARG;
  const fbl_mlp_plan* p = plan;
  const size_t n = (size_t)p->n_pad, e = (size_t)p->base->e;
  const bool gated = p->d.act == FBL_ACT_SWIGLU;
  switch (what) {
    case FBL_MWS_STATS: *offset = p->sv_stats; *bytes = n * 2 * sizeof(float); return FBL_OK;
    case FBL_MWS_XN: *offset = p->sv_xn; *bytes = n * p->d.d_model * e; return FBL_OK;
    case FBL_MWS_U: *offset = p->sv_u; *bytes = n * p->d.d_ff * e; return FBL_OK;
    case FBL_MWS_G: if (!gated) return FBL_ERR_INVALID_ARG; *offset = p->sv_g; *bytes = n * p->d.d_ff * e; return FBL_OK;
    case FBL_MWS_H: *offset = p->sv_h; *bytes = n * p->d.d_ff * e; return FBL_OK;
    case FBL_MWS_DU: *offset = p->sb_du; *bytes = n * p->d.d_ff * e; return FBL_OK;
    case FBL_MWS_DG: if (!gated) return FBL_ERR_INVALID_ARG; *offset = p->sb_dg; *bytes = n * p->d.d_ff * e; return FBL_OK;
    case FBL_MWS_DXN: *offset = p->sb_dxn; *bytes = n * p->d.d_model * e; return FBL_OK;
    default: return FBL_ERR_INVALID_ARG;
  }
}

static int mlp_pack_common(const fbl_mlp_plan* plan, int id, const void* src, void* dst, void* stream, int unpack) {
  int64_t outer, rows, rows_pad; int cols;
  if (!plan || !src || !dst || !mshape(plan, id, &outer, &rows, &rows_pad, &cols)) return FBL_ERR_INVALID_ARG;
  if (misaligned(unpack ? src : dst)) return FBL_ERR_MISALIGNED;
  MLP_CUDA(launch_pack(plan->d.dtype, unpack, src, dst, outer, rows, rows_pad, cols, as_stream(stream)));
  return FBL_OK;
}
int fbl_mlp_pack(const fbl_mlp_plan* plan, int id, const void* rowmajor_dev, void* tiled_dev, void* stream) {
  return mlp_pack_common(plan, id, rowmajor_dev, tiled_dev, stream, 0);
}
int fbl_mlp_unpack(const fbl_mlp_plan* plan, int id, const void* tiled_dev, void* rowmajor_dev, void* stream) {
  return mlp_pack_common(plan, id, tiled_dev, rowmajor_dev, stream, 1);
}

int fbl_mlp_status_poll(const fbl_mlp_plan* plan, const void* scratch, int32_t* device_status) {
  if (!plan) return FBL_ERR_INVALID_ARG;
  return fbl_status_poll(plan->base, scratch, device_status);
}

int fbl_mlp_fwd(const fbl_mlp_plan* p, const void* X, const float* gamma, const float* beta, const void* W1,
                const void* Wg, const void* W2, const float* b1, const float* bg, const float* b2, void* Y, void* saved,
                void* scratch, void* stream) {
  if (!p || !X || !gamma || !W1 || !W2 || !Y || !saved || !scratch) return FBL_ERR_INVALID_ARG;
  const bool gated = p->d.act == FBL_ACT_SWIGLU, bias = p->d.has_bias != 0;
  if (gated && !Wg) return FBL_ERR_INVALID_ARG;
  if (bias && (!b1 || !b2 || (gated && !bg))) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !beta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {X, W1, gated ? Wg : W1, W2, Y, saved, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  const fbl_plan* bp = p->base;
  char* sv = (char*)saved;
  int32_t* status = (int32_t*)scratch;
  float* stats = (float*)(sv + p->sv_stats);
  void* Xn = sv + p->sv_xn; void* U = sv + p->sv_u; void* G = sv + p->sv_g; void* H = sv + p->sv_h;
  const int n = (int)p->n_pad, D = p->d.d_model, F = p->d.d_ff;

  if (!norm_fwd_resets_status(bp)) MLP_CUDA(cudaMemsetAsync(status, 0, FBL_ALIGN, st));
  MLP_STEP(1, launch_norm_fwd(bp, X, gamma, beta, Xn, stats, status, st));
  {
    GemmArgs gs[2];
    const void* W[2] = {W1, Wg}; void* O[2] = {U, G}; const float* B[2] = {b1, bg};
    const int cnt = gated ? 2 : 1;
    bool tc = bp->use_tc != 0;
    for (int i = 0; i < cnt; ++i) {
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = n; g.n = F; g.n_terms = 1;
      g.t[0] = {Xn, p->n_pad, 0, W[i], D, 0, D};
      g.b_static = 1;
      g.c = O[i]; g.c_rpad = p->n_pad; g.bias = bias ? B[i] : nullptr;
      g.seq = p->d.seq; g.t_pad = bp->t_pad;
      tc = tc && gemm_tc_supported(bp, g);
    }
    int k = 0;
    if (tc && !gated) {
      // the activation rides in the up projection's epilogue: U and H = gelu(U) leave the same accumulator tile
      gs[0].epi = 1; gs[0].c2 = H;
      MLP_CUDA(run_group(p, gs, 1, status, st, &k));
      p->launches += k;
    } else if (tc) {
      // gated: U first, then the gate projection, whose epilogue reads U's tile and writes G and H = silu(G) * U
      MLP_CUDA(run_group(p, &gs[0], 1, status, st, &k));
      p->launches += k;
      gs[1].epi = 3; gs[1].residual = U; gs[1].c2 = H;
      MLP_CUDA(run_group(p, &gs[1], 1, status, st, &k));
      p->launches += k;
    } else {
      MLP_CUDA(run_group(p, gs, cnt, status, st, &k));
      p->launches += k;
      MLP_STEP(1, act(p, false, nullptr, U, G, H, nullptr, st));
    }
  }
  {
    GemmArgs g = {};
    g.m = n; g.n = D; g.n_terms = 1;
    g.t[0] = {H, p->n_pad, 0, W2, F, 0, F};
    g.b_static = 1;
    g.c = Y; g.c_rpad = p->n_pad; g.bias = bias ? b2 : nullptr;
    g.residual = p->d.residual ? X : nullptr;
    g.seq = p->d.seq; g.t_pad = bp->t_pad;
    int k = 0;
    MLP_CUDA(run_group(p, &g, 1, status, st, &k));
    p->launches += k;
  }
  return FBL_OK;
}

int fbl_mlp_bwd(const fbl_mlp_plan* p, const void* dY, const void* X, const float* gamma, const void* W1, const void* Wg,
                const void* W2, const void* saved, void* dX, void* dW1, void* dWg, void* dW2, float* db1, float* dbg,
                float* db2, float* dgamma, float* dbeta, void* scratch, void* stream) {
  if (!p || !dY || !X || !gamma || !W1 || !W2 || !saved || !dX || !dW1 || !dW2 || !dgamma || !scratch) return FBL_ERR_INVALID_ARG;
  const bool gated = p->d.act == FBL_ACT_SWIGLU, bias = p->d.has_bias != 0;
  if (gated && (!Wg || !dWg)) return FBL_ERR_INVALID_ARG;
  if (bias && (!db1 || !db2 || (gated && !dbg))) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !dbeta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {dY, X, W1, gated ? Wg : W1, W2, saved, dX, dW1, gated ? dWg : dW1, dW2, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  const fbl_plan* bp = p->base;
  const char* sv = (const char*)saved;
  char* sc = (char*)scratch;
  int32_t* status = (int32_t*)sc;
  const float* stats = (const float*)(sv + p->sv_stats);
  const void* Xn = sv + p->sv_xn; const void* U = sv + p->sv_u; const void* G = sv + p->sv_g; const void* H = sv + p->sv_h;
  void* dH = sc + p->sb_dh; void* dU = sc + p->sb_du; void* dG = sc + p->sb_dg; void* dXn = sc + p->sb_dxn;
  float* part = (float*)(sc + p->sb_part);
  const int n = (int)p->n_pad, D = p->d.d_model, F = p->d.d_ff;
  const bool tc = bp->use_tc != 0;
  const bool split2 = tc && p->ksplit_2 > 1, split1 = tc && p->ksplit_1 > 1;

  MLP_CUDA(cudaMemsetAsync(status, 0, p->zero_bytes, st));     // status word + accumulation areas of sliced reductions
  ConvertGroup cg = {};
  {
    GemmArgs gs[2];
    GemmArgs& gw = gs[0];     // dW2 = H^T dY : token-axis reduction, H's tiles read MN-major
    gw = GemmArgs{};
    gw.m = F; gw.n = D; gw.n_terms = 1;
    gw.t[0] = {H, p->n_pad, 1, dY, p->n_pad, 0, n};
    gw.c = dW2; gw.c_rpad = up8(F);
    GemmArgs& gh = gs[1];     // dH = dY W2^T : W2's tiles read with the roles of its axes swapped
    gh = GemmArgs{};
    gh.m = n; gh.n = F; gh.n_terms = 1;
    gh.t[0] = {dY, p->n_pad, 0, W2, F, 1, D};
    gh.b_static = 1;
    gh.c = dH; gh.c_rpad = p->n_pad; gh.seq = p->d.seq; gh.t_pad = bp->t_pad;
    bool both_tc = tc && gemm_tc_supported(bp, gw) && gemm_tc_supported(bp, gh);
    if (split2 && both_tc) {
      gw.ksplit = p->ksplit_2; gw.acc = (float*)(sc + p->sb_acc2);
      cg.src[cg.count] = gw.acc; cg.dst[cg.count] = dW2; cg.n[cg.count] = up8(F) * (int64_t)D; cg.count++;
    }
    int k = 0;
    if (both_tc) {
      // the activation's derivative rides in the dH product's epilogue: dU (and dG) leave the accumulator tile, dH
      // itself is never stored
      gh.epi = gated ? 4 : 2; gh.residual = U; gh.aux1 = gated ? G : nullptr; gh.c = dU; gh.c2 = gated ? dG : nullptr;
      MLP_CUDA(run_group(p, gs, 2, status, st, &k));
      p->launches += k;
    } else {
      MLP_CUDA(run_group(p, gs, 2, status, st, &k));
      p->launches += k;
      MLP_STEP(1, act(p, true, dH, U, G, dU, dG, st));
    }
  }
  {
    GemmArgs gs[3];
    const void* Gr[2] = {dU, dG}; void* DW[2] = {dW1, dWg};
    const int nw = gated ? 2 : 1;
    bool all_tc = tc;
    for (int i = 0; i < nw; ++i) {      // dW1 = Xn^T dU (dWg = Xn^T dG): token-axis reductions
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = D; g.n = F; g.n_terms = 1;
      g.t[0] = {Xn, p->n_pad, 1, Gr[i], p->n_pad, 0, n};
      g.c = DW[i]; g.c_rpad = up8(D);
      all_tc = all_tc && gemm_tc_supported(bp, g);
    }
    GemmArgs& gx = gs[nw];              // dXn = dU W1^T (+ dG Wg^T): one accumulator, one or two reduction loops
    gx = GemmArgs{};
    gx.m = n; gx.n = D; gx.n_terms = nw;
    gx.t[0] = {dU, p->n_pad, 0, W1, D, 1, F};
    gx.b_static = 1;
    if (gated) gx.t[1] = {dG, p->n_pad, 0, Wg, D, 1, F};
    gx.c = dXn; gx.c_rpad = p->n_pad; gx.seq = p->d.seq; gx.t_pad = bp->t_pad;
    all_tc = all_tc && gemm_tc_supported(bp, gx);
    if (split1 && all_tc) {
      float* acc = (float*)(sc + p->sb_acc1);
      for (int i = 0; i < nw; ++i) {
        gs[i].ksplit = p->ksplit_1; gs[i].acc = acc;
        cg.src[cg.count] = acc; cg.dst[cg.count] = DW[i]; cg.n[cg.count] = up8(D) * (int64_t)F; cg.count++;
        acc += up8(D) * (int64_t)F;
      }
    }
    int k = 0;
    MLP_CUDA(run_group(p, gs, nw + 1, status, st, &k));
    p->launches += k;
  }
  if (cg.count > 0) MLP_STEP(1, launch_convert_f32_group(cg, st));
  // bias gradients: token-axis column sums of dY, dU (and dG), sharing the norm backward's launches where they can
  const void* M3[3] = {dY, dU, dG};
  float* O3[3] = {db2, db1, dbg};
  const int C3[3] = {D, F, F};
  const int nb = gated ? 3 : 2;
  if (bias && norm_bwd_takes_colsums(bp)) {
    MLP_STEP(2, launch_norm_bwd(bp, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, part, st, nb, M3, C3, O3));
    return FBL_OK;
  }
  if (bias) MLP_STEP(2, launch_colsum_group(p->d.dtype, nb, M3, p->n_pad, C3, O3, part, st));
  MLP_STEP(norm_bwd_takes_colsums(bp) ? 2 : 1, launch_norm_bwd(bp, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, part, st));
  return FBL_OK;
}

}  // extern "C"
