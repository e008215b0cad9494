// C ABI: plan construction, the host-side integer index maps, and the forward/backward drivers.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "fbl_internal.h"

namespace {

inline int64_t up8(int64_t v) { return (v + 7) / 8 * 8; }

struct MatShape { int64_t outer, rows, rows_pad; int cols; };   // rows_pad per outer slice

bool mat_shape(const fbl_plan* p, int id, MatShape* s) {
  const fbl_layer_desc& d = p->d;
  switch (id) {
    case FBL_T_X: case FBL_T_Y: case FBL_T_DY: case FBL_T_DX: case FBL_T_XN:
      *s = {d.batch, d.seq, p->t_pad, d.d_model}; return true;
    case FBL_T_Q: case FBL_T_A: case FBL_T_Q_HEADS: case FBL_T_A_HEADS:
      *s = {d.batch, d.seq, p->t_pad, p->dq}; return true;
    case FBL_T_K: case FBL_T_V: case FBL_T_K_HEADS: case FBL_T_V_HEADS:
      *s = {d.batch, p->seq_kv, p->t_pad_kv, p->dkv}; return true;
    case FBL_T_MEM: case FBL_T_DMEM:
      if (!p->cross) return false;
      *s = {d.batch, p->seq_kv, p->t_pad_kv, p->d_mem}; return true;
    case FBL_T_WQ: case FBL_T_WQ_T: *s = {1, d.d_model, up8(d.d_model), p->dq}; return true;
    case FBL_T_WK: case FBL_T_WV: case FBL_T_WK_T: case FBL_T_WV_T:
      *s = {1, p->d_mem, up8(p->d_mem), p->dkv}; return true;
    case FBL_T_WO: case FBL_T_WO_T: *s = {1, p->dq, up8(p->dq), d.d_model}; return true;
    default: return false;
  }
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & (FBL_ALIGN - 1)) != 0; }

thread_local char g_detail[256] = "";

#define FBL_CUDA(expr)                                  \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) {                           \
      fbl_note_cuda_error(e__, #expr);                  \
      return FBL_ERR_CUDA;                              \
    }                                                   \
  } while (0)

// One named step of a driver: launch, count the kernels it enqueued, and (when profiling is on) record an
// event after it so the per-step device time can be read back later.
#define FBL_STEP(name, kernels, expr)                              \
  do {                                                             \
    FBL_CUDA(expr);                                                \
    const fbl_plan* mp__ = p;                                      \
    mp__->launches += (kernels);                                   \
    if (mp__->prof_on && mp__->prof_n < FBL_PROF_MAX) {            \
      mp__->prof_name[mp__->prof_n] = (name);                      \
      FBL_CUDA(cudaEventRecord(mp__->prof_ev[1 + mp__->prof_n], st)); \
      mp__->prof_n++;                                              \
    }                                                              \
  } while (0)

#define FBL_PROF_BEGIN()                                           \
  do {                                                             \
    const fbl_plan* mp__ = p;                                      \
    if (mp__->prof_on) { mp__->prof_n = 0; FBL_CUDA(cudaEventRecord(mp__->prof_ev[0], st)); } \
  } while (0)

cudaError_t run_gemm(const fbl_plan* p, const GemmArgs& g, int32_t* status, cudaStream_t st, int launch_id = -1) {
  if (p->use_tc && gemm_tc_supported(p, g)) return launch_gemm_tc_group(p, &g, 1, status, st, launch_id);
  return launch_gemm_simt(p->d.dtype, g, st);
}

}  // namespace

void fbl_note_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_detail, sizeof(g_detail), "%s: %s", cudaGetErrorString(e), where);
}

extern "C" {

const char* fbl_last_error_detail(void) { return g_detail; }

// Shared by the two plan constructors.  cross = 0: self-attention (the key side is the layer's own sequence);
// cross = 1: K and V are projected from a memory [batch, seq_kv, d_mem].
static int plan_build(const fbl_layer_desc* desc, int cross, int seq_kv_in, int d_mem_in, fbl_plan** out) {
  if (!desc || !out) return FBL_ERR_INVALID_ARG;
  *out = nullptr;
  const fbl_layer_desc& d = *desc;
  const int seq_kv = cross ? seq_kv_in : d.seq, d_mem = cross ? d_mem_in : d.d_model;
  if (cross && (seq_kv <= 0 || d_mem <= 0)) return FBL_ERR_INVALID_ARG;
  if (cross && d.causal) return FBL_ERR_INVALID_ARG;      // memory positions have no order relative to the queries
  if (d.batch <= 0 || d.seq <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.head_dim <= 0)
    return FBL_ERR_INVALID_ARG;
  if (d.dtype != FBL_DTYPE_FP32 && d.dtype != FBL_DTYPE_BF16) return FBL_ERR_INVALID_ARG;
  if (d.norm != FBL_NORM_LAYERNORM && d.norm != FBL_NORM_RMSNORM) return FBL_ERR_INVALID_ARG;
  if (!(d.eps >= 0.f)) return FBL_ERR_INVALID_ARG;
  const int e = d.dtype == FBL_DTYPE_FP32 ? 4 : 2;
  const int tw = 128 / e;
  // Tile-propagation legality (section 4.3): the GQA head map needs whole groups; the head split
  // must fall on tile boundaries (tile_w divides head_dim) and d_model must be whole tiles.
  if (d.n_q_heads % d.n_kv_heads != 0) return FBL_ERR_UNSUPPORTED_SHAPE;
  if (d.head_dim % tw != 0 || d.d_model % tw != 0 || d_mem % tw != 0) return FBL_ERR_UNSUPPORTED_SHAPE;
  if (d.dtype == FBL_DTYPE_FP32 && d.head_dim != 32 && d.head_dim != 64 && d.head_dim != 128)
    return FBL_ERR_UNSUPPORTED_SHAPE;
  if (d.dtype == FBL_DTYPE_BF16 && d.head_dim != 64 && d.head_dim != 128) return FBL_ERR_UNSUPPORTED_SHAPE;
  if ((int64_t)d.batch * up8(d.seq) > (int64_t)1 << 30) return FBL_ERR_UNSUPPORTED_SHAPE;
  if ((int64_t)d.batch * up8(seq_kv) > (int64_t)1 << 30) return FBL_ERR_UNSUPPORTED_SHAPE;
  if (d.d_model > 16384 || d_mem > 16384 || (int64_t)d.n_q_heads * d.head_dim > 16384) return FBL_ERR_UNSUPPORTED_SHAPE;

  fbl_plan* p = new (std::nothrow) fbl_plan();
  if (!p) return FBL_ERR_INVALID_ARG;
  p->d = d;
  p->e = e;
  p->tw = tw;
  p->t_pad = (int)up8(d.seq);
  p->n_pad = (int64_t)d.batch * p->t_pad;
  p->cross = cross;
  p->seq_kv = seq_kv;
  p->d_mem = d_mem;
  p->t_pad_kv = (int)up8(seq_kv);
  p->n_pad_kv = (int64_t)d.batch * p->t_pad_kv;
  p->dq = d.n_q_heads * d.head_dim;
  p->dkv = d.n_kv_heads * d.head_dim;
  p->group = d.n_q_heads / d.n_kv_heads;
  p->scale = d.softmax_scale > 0.f ? d.softmax_scale : 1.0f / sqrtf((float)d.head_dim);
  // SM count of the current device; a host without a device (index-map and sizing calls only) plans for 148 SMs
  p->sm_count = 148;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      p->sm_count = sms;
    else
      (void)cudaGetLastError();       // no device: not an error of this call
  }
  auto env_int = [](const char* name, int dflt) { const char* v = getenv(name); return v ? atoi(v) : dflt; };
  p->knob_gemm_pair = env_int("FBL_GEMM_PAIR", -1);
  p->knob_gemm_esets = env_int("FBL_GEMM_ESETS", 0);
  p->knob_fwd_tiles = env_int("FBL_FWD_TILES", 0);
  for (int i = 0; i < FBL_GEMM_LAUNCH_COUNT; ++i) p->choice[i] = {0, -1, 0};
  p->use_tc = d.dtype == FBL_DTYPE_BF16 ? 1 : 0;

  const size_t n = (size_t)p->n_pad, nk = (size_t)p->n_pad_kv;
  auto mat = [&](size_t cols) { return fbl_align_up(n * cols * (size_t)e, FBL_ALIGN); };
  auto mat_kv = [&](size_t cols) { return fbl_align_up(nk * cols * (size_t)e, FBL_ALIGN); };
  const size_t rows_bh = (size_t)d.batch * d.n_q_heads * p->t_pad;
  size_t o = 0;
  p->sv_stats = o; o += fbl_align_up(n * 2 * sizeof(float), FBL_ALIGN);
  p->sv_xn = o;    o += mat(d.d_model);
  p->sv_q = o;     o += mat(p->dq);
  p->sv_k = o;     o += mat_kv(p->dkv);
  p->sv_v = o;     o += mat_kv(p->dkv);
  p->sv_a = o;     o += mat(p->dq);
  p->sv_lse = o;   o += fbl_align_up(rows_bh * sizeof(float) + 512, FBL_ALIGN);   // + one 128-float copy window past the last row
  p->saved_bytes = o;

  // Partial-sum area of the backward's token-axis reductions: the slab partials of the four bias column sums
  // first, then (from the next 256-float boundary) the norm backward's per-block partial rows, at most two
  // blocks per SM with one dgamma row and one dbeta row each.
  {
    const size_t cs_floats = colsum_scratch_bytes(p->n_pad, (int64_t)d.d_model + p->dq + (cross ? 0 : 2 * p->dkv)) / sizeof(float);
    const size_t norm_floats = (size_t)2 * p->sm_count * 2 * d.d_model;
    p->part_bytes = fbl_align_up(((cs_floats + 255) / 256 * 256 + norm_floats) * sizeof(float), FBL_ALIGN);
  }

  p->scratch_fwd_bytes = FBL_ALIGN;  // the status word

  // weight-gradient GEMMs: few output tiles, reduction over all tokens; slice the reduction when that balances the SMs
  p->ksplit_o = p->ksplit_qkv = p->ksplit_kv = 1;
  if (p->use_tc && cross) {
    const int kb_q = (int)((p->n_pad + 63) / 64), kb_k = (int)((p->n_pad_kv + 63) / 64);
    const GemmShape go[2] = {{p->dq, d.d_model, kb_q, 1}, {p->n_pad, p->dq, (d.d_model + 63) / 64, 0}};
    p->ksplit_o = gemm_tc_choose_split(p->sm_count, go, 2);
    const GemmShape gq[2] = {{d.d_model, p->dq, kb_q, 1}, {p->n_pad, d.d_model, (p->dq + 63) / 64, 0}};
    p->ksplit_qkv = gemm_tc_choose_split(p->sm_count, gq, 2);
    const GemmShape gk[3] = {{d_mem, p->dkv, kb_k, 1}, {d_mem, p->dkv, kb_k, 1}, {p->n_pad_kv, d_mem, (2 * p->dkv + 63) / 64, 0}};
    p->ksplit_kv = gemm_tc_choose_split(p->sm_count, gk, 3);
  } else if (p->use_tc) {
    const int kb_tok = (int)((p->n_pad + 63) / 64);
    const GemmShape go[2] = {{p->dq, d.d_model, kb_tok, 1}, {p->n_pad, p->dq, (d.d_model + 63) / 64, 0}};
    p->ksplit_o = gemm_tc_choose_split(p->sm_count, go, 2);
    const GemmShape gq[4] = {{d.d_model, p->dq, kb_tok, 1}, {d.d_model, p->dkv, kb_tok, 1}, {d.d_model, p->dkv, kb_tok, 1},
                             {p->n_pad, d.d_model, (p->dq + 2 * p->dkv + 63) / 64, 0}};
    p->ksplit_qkv = gemm_tc_choose_split(p->sm_count, gq, 4);
  }
  if (p->use_tc && getenv("FBL_KSPLIT_O")) p->ksplit_o = atoi(getenv("FBL_KSPLIT_O"));          // tuning knobs
  if (p->use_tc && getenv("FBL_KSPLIT_QKV")) p->ksplit_qkv = atoi(getenv("FBL_KSPLIT_QKV"));
  if (getenv("FBL_VERBOSE")) fprintf(stderr, "fblayout: reduction slices dWo %d, dWq/dWk/dWv %d\n", p->ksplit_o, p->ksplit_qkv);
  o = FBL_ALIGN;  // status word, then the fp32 accumulation areas
  p->sb_acc_o = o;
  if (p->ksplit_o > 1) o += fbl_align_up((size_t)up8(p->dq) * d.d_model * sizeof(float), FBL_ALIGN);
  p->sb_acc_qkv = o;
  if (p->ksplit_qkv > 1) o += fbl_align_up((size_t)up8(d.d_model) * (p->dq + (cross ? 0 : 2 * p->dkv)) * sizeof(float), FBL_ALIGN);
  p->sb_acc_kv = o;
  if (cross && p->ksplit_kv > 1) o += fbl_align_up((size_t)up8(d_mem) * 2 * p->dkv * sizeof(float), FBL_ALIGN);
  p->acc_bytes = o - FBL_ALIGN;
  p->sb_dqacc = o; o += fbl_align_up(n * p->dq * sizeof(float), FBL_ALIGN);   // zero-filled with the areas before it
  p->zero_bytes = o;
  p->sb_da = o;    o += mat(p->dq);
  p->sb_dvec = o;  o += fbl_align_up(rows_bh * sizeof(float), FBL_ALIGN);
  p->sb_dq = o;    o += mat(p->dq);
  p->sb_dk = o;    o += mat_kv(p->dkv);
  p->sb_dv = o;    o += mat_kv(p->dkv);
  p->sb_dxn = o;   o += mat(d.d_model);
  p->sb_part = o;  o += p->part_bytes;
  p->sb_part_kv = o;
  if (cross) o += fbl_align_up(colsum_scratch_bytes(p->n_pad_kv, 2 * (int64_t)p->dkv), FBL_ALIGN);
  p->scratch_bwd_bytes = o;
  *out = p;
  return FBL_OK;
}

int fbl_plan_create(const fbl_layer_desc* desc, fbl_plan** out) { return plan_build(desc, 0, 0, 0, out); }

int fbl_xattn_plan_create(const fbl_layer_desc* desc, int32_t seq_kv, int32_t d_mem, fbl_plan** out) {
  return plan_build(desc, 1, seq_kv, d_mem, out);
}

void fbl_plan_destroy(fbl_plan* plan) {
  if (!plan) return;
  if (plan->prof_on)
    for (int i = 0; i <= FBL_PROF_MAX; ++i) cudaEventDestroy(plan->prof_ev[i]);
  delete plan;
}

int fbl_profile_enable(fbl_plan* plan, int enable) {
  if (!plan) return FBL_ERR_INVALID_ARG;
  if (enable && !plan->prof_on) {
    for (int i = 0; i <= FBL_PROF_MAX; ++i) FBL_CUDA(cudaEventCreate(&plan->prof_ev[i]));
    plan->prof_on = 1;
  } else if (!enable && plan->prof_on) {
    for (int i = 0; i <= FBL_PROF_MAX; ++i) cudaEventDestroy(plan->prof_ev[i]);
    plan->prof_on = 0;
  }
  plan->prof_n = 0;
  return FBL_OK;
}

int fbl_profile_read(const fbl_plan* plan, int max_steps, const char** names, float* ms) {
  if (!plan || !names || !ms || !plan->prof_on) return FBL_ERR_INVALID_ARG;
  int n = plan->prof_n < max_steps ? plan->prof_n : max_steps;
  for (int i = 0; i < n; ++i) {
    names[i] = plan->prof_name[i];
    FBL_CUDA(cudaEventElapsedTime(&ms[i], plan->prof_ev[i], plan->prof_ev[i + 1]));
  }
  return n;
}

int64_t fbl_launch_count(const fbl_plan* plan) { return plan ? plan->launches : -1; }

int fbl_plan_set_gemm_choice(fbl_plan* plan, int launch_id, int tile_n, int cta_pair, int epilogue_sets) {
  if (!plan || launch_id < 0 || launch_id >= FBL_GEMM_LAUNCH_COUNT) return FBL_ERR_INVALID_ARG;
  if ((tile_n != 0 && tile_n != 128 && tile_n != 256) || cta_pair < -1 || cta_pair > 1 || epilogue_sets < 0 || epilogue_sets > 2)
    return FBL_ERR_INVALID_ARG;
  plan->choice[launch_id] = {tile_n, cta_pair, epilogue_sets};
  return FBL_OK;
}

int fbl_plan_enable_rope(fbl_plan* plan, float base) {
  if (!plan || plan->cross || !(base > 1.f) || plan->d.head_dim % 16 != 0) return FBL_ERR_INVALID_ARG;
  plan->rope_base = base;
  return FBL_OK;
}

int fbl_plan_set_kernel_path(fbl_plan* plan, int path) {
  if (!plan || (path != 0 && path != 1)) return FBL_ERR_INVALID_ARG;
  plan->use_tc = (path == 0 && plan->d.dtype == FBL_DTYPE_BF16) ? 1 : 0;
  return FBL_OK;
}

int fbl_tensor_bytes(const fbl_plan* plan, int tensor_id, size_t* bytes) {
  MatShape s;
  if (!plan || !bytes || !mat_shape(plan, tensor_id, &s)) return FBL_ERR_INVALID_ARG;
  *bytes = (size_t)(s.outer * s.rows_pad) * s.cols * plan->e;
  return FBL_OK;
}

int fbl_workspace_bytes(const fbl_plan* plan, size_t* saved, size_t* scratch_fwd, size_t* scratch_bwd) {
  if (!plan) return FBL_ERR_INVALID_ARG;
  if (saved) *saved = plan->saved_bytes;
  if (scratch_fwd) *scratch_fwd = plan->scratch_fwd_bytes;
  if (scratch_bwd) *scratch_bwd = plan->scratch_bwd_bytes;
  return FBL_OK;
}

int fbl_workspace_offset(const fbl_plan* plan, int what, size_t* offset, size_t* bytes) {
  if (!plan || !offset || !bytes) return FBL_ERR_INVALID_ARG;
  const fbl_plan* p = plan;
  const size_t n = (size_t)p->n_pad, nk = (size_t)p->n_pad_kv, e = (size_t)p->e;
  const size_t rows_bh = (size_t)p->d.batch * p->d.n_q_heads * p->t_pad;
  switch (what) {
    case FBL_WS_STATS: *offset = p->sv_stats; *bytes = n * 2 * sizeof(float); return FBL_OK;
    case FBL_WS_XN: *offset = p->sv_xn; *bytes = n * p->d.d_model * e; return FBL_OK;
    case FBL_WS_Q: *offset = p->sv_q; *bytes = n * p->dq * e; return FBL_OK;
    case FBL_WS_K: *offset = p->sv_k; *bytes = nk * p->dkv * e; return FBL_OK;
    case FBL_WS_V: *offset = p->sv_v; *bytes = nk * p->dkv * e; return FBL_OK;
    case FBL_WS_A: *offset = p->sv_a; *bytes = n * p->dq * e; return FBL_OK;
    case FBL_WS_LSE: *offset = p->sv_lse; *bytes = rows_bh * sizeof(float); return FBL_OK;
    case FBL_WS_D: *offset = p->sb_dvec; *bytes = rows_bh * sizeof(float); return FBL_OK;
    case FBL_WS_DA: *offset = p->sb_da; *bytes = n * p->dq * e; return FBL_OK;
    case FBL_WS_DQ: *offset = p->sb_dq; *bytes = n * p->dq * e; return FBL_OK;
    case FBL_WS_DK: *offset = p->sb_dk; *bytes = nk * p->dkv * e; return FBL_OK;
    case FBL_WS_DV: *offset = p->sb_dv; *bytes = nk * p->dkv * e; return FBL_OK;
    case FBL_WS_DXN: *offset = p->sb_dxn; *bytes = n * p->d.d_model * e; return FBL_OK;
    case FBL_WS_PARTIALS: *offset = p->sb_part; *bytes = p->part_bytes; return FBL_OK;
    default: return FBL_ERR_INVALID_ARG;
  }
}

int64_t fbl_tile_offset(const fbl_plan* plan, int tensor_id, const int32_t idx[4]) {
  MatShape s;
  if (!plan || !idx || !mat_shape(plan, tensor_id, &s)) return -1;
  const fbl_layer_desc& d = plan->d;
  int64_t r, c;
  switch (tensor_id) {
    case FBL_T_Q_HEADS: case FBL_T_A_HEADS: case FBL_T_K_HEADS: case FBL_T_V_HEADS: {
      const int heads = (tensor_id == FBL_T_K_HEADS || tensor_id == FBL_T_V_HEADS) ? d.n_kv_heads : d.n_q_heads;
      if (idx[0] < 0 || idx[0] >= d.batch || idx[1] < 0 || idx[1] >= heads || idx[2] < 0 || idx[2] >= s.rows ||
          idx[3] < 0 || idx[3] >= d.head_dim) return -1;
      r = (int64_t)idx[0] * s.rows_pad + idx[2];
      c = (int64_t)idx[1] * d.head_dim + idx[3];
      break;
    }
    case FBL_T_WQ_T: case FBL_T_WK_T: case FBL_T_WV_T: case FBL_T_WO_T:
      if (idx[0] < 0 || idx[0] >= s.cols || idx[1] < 0 || idx[1] >= s.rows) return -1;
      r = idx[1]; c = idx[0];
      break;
    case FBL_T_WQ: case FBL_T_WK: case FBL_T_WV: case FBL_T_WO:
      if (idx[0] < 0 || idx[0] >= s.rows || idx[1] < 0 || idx[1] >= s.cols) return -1;
      r = idx[0]; c = idx[1];
      break;
    default:
      if (idx[0] < 0 || idx[0] >= s.outer || idx[1] < 0 || idx[1] >= s.rows || idx[2] < 0 || idx[2] >= s.cols)
        return -1;
      r = (int64_t)idx[0] * s.rows_pad + idx[1];
      c = idx[2];
  }
  return rt_off_dyn(plan->tw, s.outer * s.rows_pad, r, c);
}

int fbl_tile_map(const fbl_plan* plan, int map_id, int64_t src, int64_t* dst) {
  if (!plan || !dst || src < 0) return FBL_ERR_INVALID_ARG;
  const fbl_layer_desc& d = plan->d;
  const int64_t rt = plan->n_pad / 8;            // row tiles of a token matrix
  const int64_t st = plan->t_pad / 8;            // row tiles per sequence
  const int64_t hw = d.head_dim / plan->tw;      // tiles across one head
  switch (map_id) {
    case FBL_MAP_SPLIT_Q: case FBL_MAP_SPLIT_KV: case FBL_MAP_MERGE_Q: case FBL_MAP_MERGE_KV: {
      const int64_t heads = (map_id == FBL_MAP_SPLIT_Q || map_id == FBL_MAP_MERGE_Q) ? d.n_q_heads : d.n_kv_heads;
      const int64_t ct = heads * hw;
      if (src >= rt * ct) return FBL_ERR_INVALID_ARG;
      if (map_id == FBL_MAP_SPLIT_Q || map_id == FBL_MAP_SPLIT_KV) {
        // f = (transpose S<->H) o (reshape D -> H x HD), on tile coordinates; the inner modulo chain
        // (src mod ct) mod hw collapses to src mod hw because hw divides ct (the paper's identity).
        const int64_t tr = src / ct, td = src % hw, h = (src % ct) / hw;
        const int64_t b = tr / st, ts = tr % st;
        *dst = ((b * heads + h) * st + ts) * hw + td;
      } else {
        const int64_t td = src % hw, ts = (src / hw) % st, bh = src / (hw * st);
        const int64_t b = bh / heads, h = bh % heads;
        *dst = (b * st + ts) * ct + h * hw + td;
      }
      return FBL_OK;
    }
    case FBL_MAP_TRANSPOSE_WQ: case FBL_MAP_TRANSPOSE_WO: {
      const int64_t rows = map_id == FBL_MAP_TRANSPOSE_WQ ? d.d_model : plan->dq;
      const int64_t cols = map_id == FBL_MAP_TRANSPOSE_WQ ? plan->dq : d.d_model;
      const int64_t trs = up8(rows) / 8, tcs = cols / plan->tw;
      if (src >= trs * tcs) return FBL_ERR_INVALID_ARG;
      *dst = (src % tcs) * trs + src / tcs;
      return FBL_OK;
    }
    case FBL_MAP_PHYS_Q: {
      const int64_t ct = d.n_q_heads * hw;
      if (src >= rt * ct) return FBL_ERR_INVALID_ARG;
      *dst = (src % ct) * rt + src / ct;
      return FBL_OK;
    }
    case FBL_MAP_PHYS_WQ: {
      const int64_t trs = up8(d.d_model) / 8, tcs = plan->dq / plan->tw;
      if (src >= trs * tcs) return FBL_ERR_INVALID_ARG;
      *dst = (src % tcs) * trs + src / tcs;
      return FBL_OK;
    }
    default: return FBL_ERR_INVALID_ARG;
  }
}

static int pack_common(const fbl_plan* plan, int tensor_id, const void* src, void* dst, void* stream, int unpack) {
  MatShape s;
  if (!plan || !src || !dst || !mat_shape(plan, tensor_id, &s)) return FBL_ERR_INVALID_ARG;
  if (tensor_id >= FBL_T_Q_HEADS && tensor_id <= FBL_T_WO_T) return FBL_ERR_INVALID_ARG;   // views are not separate buffers
  if (misaligned(unpack ? src : dst)) return FBL_ERR_MISALIGNED;
  FBL_CUDA(launch_pack(plan->d.dtype, unpack, src, dst, s.outer, s.rows, s.rows_pad, s.cols, as_stream(stream)));
  return FBL_OK;
}
int fbl_pack(const fbl_plan* plan, int tensor_id, const void* rowmajor_dev, void* tiled_dev, void* stream) {
  return pack_common(plan, tensor_id, rowmajor_dev, tiled_dev, stream, 0);
}
int fbl_unpack(const fbl_plan* plan, int tensor_id, const void* tiled_dev, void* rowmajor_dev, void* stream) {
  return pack_common(plan, tensor_id, tiled_dev, rowmajor_dev, stream, 1);
}

int fbl_layer_fwd(const fbl_plan* p, const void* X, const float* gamma, const float* beta, const void* Wq,
                  const void* Wk, const void* Wv, const void* Wo, const float* bq, const float* bk, const float* bv,
                  const float* bo, void* Y, void* saved, void* scratch, void* stream) {
  if (!p || !X || !gamma || !Wq || !Wk || !Wv || !Wo || !Y || !saved || !scratch) return FBL_ERR_INVALID_ARG;
  if (p->cross) return FBL_ERR_INVALID_ARG;              // a cross-attention plan runs through fbl_xattn_fwd / _bwd
  if (p->d.has_bias && (!bq || !bk || !bv || !bo)) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !beta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {X, Wq, Wk, Wv, Wo, Y, saved, scratch};
  for (const void* q : ptrs) if (misaligned(q)) return FBL_ERR_MISALIGNED;
  cudaStream_t st = as_stream(stream);
  char* sv = (char*)saved;
  char* sc = (char*)scratch;
  int32_t* status = (int32_t*)sc;
  float* stats = (float*)(sv + p->sv_stats);
  void* Xn = sv + p->sv_xn; void* Q = sv + p->sv_q; void* K = sv + p->sv_k; void* V = sv + p->sv_v;
  void* A = sv + p->sv_a; float* lse = (float*)(sv + p->sv_lse);
  const bool bias = p->d.has_bias;
  const int n = (int)p->n_pad, D = p->d.d_model;

  if (!norm_fwd_resets_status(p)) FBL_CUDA(cudaMemsetAsync(status, 0, FBL_ALIGN, st));
  FBL_PROF_BEGIN();
  FBL_STEP("norm_fwd", 1, launch_norm_fwd(p, X, gamma, beta, Xn, stats, status, st));
  {
    const void* W[3] = {Wq, Wk, Wv};
    void* O[3] = {Q, K, V};
    const float* B[3] = {bq, bk, bv};
    const int cols[3] = {p->dq, p->dkv, p->dkv};
    GemmArgs gs[3];
    bool tc = p->use_tc != 0;
    for (int i = 0; i < 3; ++i) {
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = n; g.n = cols[i]; g.n_terms = 1;
      g.t[0] = {Xn, p->n_pad, 0, W[i], D, 0, D};
      g.b_static = 1;
      g.c = O[i]; g.c_rpad = p->n_pad; g.bias = bias ? B[i] : nullptr;
      g.seq = p->d.seq; g.t_pad = p->t_pad;
      tc = tc && gemm_tc_supported(p, g);
    }
    if (tc) {
      FBL_STEP("proj_qkv", 1, launch_gemm_tc_group(p, gs, 3, status, st, FBL_GEMM_PROJ_QKV));   // one launch, blockIdx.z picks Q, K or V
    } else {
      for (int i = 0; i < 3; ++i)
        FBL_STEP(i == 0 ? "proj_q" : i == 1 ? "proj_k" : "proj_v", 1, launch_gemm_simt(p->d.dtype, gs[i], st));
    }
  }
  if (p->rope_base > 0.f) FBL_STEP("rope", 1, launch_rope(p, Q, p->d.n_q_heads, K, p->d.n_kv_heads, 0, st));
  if (p->use_tc && attn_fwd_tc_supported(p)) FBL_STEP("attn_fwd", 1, launch_attn_fwd_tc(p, Q, K, V, A, lse, status, st));
  else FBL_STEP("attn_fwd", 1, launch_attn_fwd_simt(p, Q, K, V, A, lse, st));
  {
    GemmArgs g = {};
    g.m = n; g.n = D; g.n_terms = 1;
    g.t[0] = {A, p->n_pad, 0, Wo, p->dq, 0, p->dq};
    g.b_static = 1;
    g.c = Y; g.c_rpad = p->n_pad; g.bias = bias ? bo : nullptr;
    g.residual = p->d.residual ? X : nullptr;
    g.seq = p->d.seq; g.t_pad = p->t_pad;
    FBL_STEP("proj_o", 1, run_gemm(p, g, status, st, FBL_GEMM_PROJ_O));
  }
  return FBL_OK;
}

int fbl_layer_bwd(const fbl_plan* p, const void* dY, const void* X, const float* gamma, const void* Wq,
                  const void* Wk, const void* Wv, const void* Wo, const void* saved, void* dX, void* dWq, void* dWk,
                  void* dWv, void* dWo, float* dbq, float* dbk, float* dbv, float* dbo, float* dgamma, float* dbeta,
                  void* scratch, void* stream) {
  if (!p || !dY || !X || !gamma || !Wq || !Wk || !Wv || !Wo || !saved || !dX || !dWq || !dWk || !dWv || !dWo ||
      !dgamma || !scratch)
    return FBL_ERR_INVALID_ARG;
  if (p->cross) return FBL_ERR_INVALID_ARG;
  if (p->d.has_bias && (!dbq || !dbk || !dbv || !dbo)) return FBL_ERR_INVALID_ARG;
  if (p->d.norm == FBL_NORM_LAYERNORM && !dbeta) return FBL_ERR_INVALID_ARG;
  const void* ptrs[] = {dY, X, Wq, Wk, Wv, Wo, saved, dX, dWq, dWk, dWv, dWo, scratch};
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
  void* part = sc + p->sb_part;
  const bool bias = p->d.has_bias;
  const int n = (int)p->n_pad, D = p->d.d_model;

  // One fill zeroes the status word and, behind it, every fp32 area the step adds into: the accumulation areas
  // of sliced weight-gradient GEMMs and the dQ accumulator.  No fill then separates later kernels of the step,
  // so each can start (programmatic dependent launch) while its predecessor drains.
  const bool split_o = p->use_tc && p->ksplit_o > 1, split_qkv = p->use_tc && p->ksplit_qkv > 1;
  // Without sliced GEMMs on the tensor-core path (only the dQ accumulator and the status word to clear) the first
  // GEMM launch does it instead: its idle epilogue warps zero the accumulator while its first tiles are computed.
  // The fill node was also the barrier between the forward and the backward kernels, which the attention backward
  // relies on when it requests forward-pass data (K, V, Q, LSE) before waiting for the kernel in front of it: that
  // GEMM is therefore launched without programmatic overlap, i.e. only once the forward pass has completed.
  bool first_gemm_fills = false;
  // (Measured: 2 % on workload 2; for accumulators of tens of MB the stores delay the launch's own first tiles by
  // more than the fill node costs, so large plans keep the node.)
  if (p->use_tc && p->acc_bytes == 0 && attn_bwd_tc_supported(p) && p->zero_bytes - p->sb_dqacc <= ((size_t)16 << 20)) {
    GemmArgs gw = GemmArgs{}, ga = GemmArgs{};
    gw.m = p->dq; gw.n = D; gw.n_terms = 1; gw.t[0] = {A, p->n_pad, 1, dY, p->n_pad, 0, n}; gw.c = dWo; gw.c_rpad = p->dq;
    ga.m = n; ga.n = p->dq; ga.n_terms = 1; ga.t[0] = {dY, p->n_pad, 0, Wo, p->dq, 1, D}; ga.c = dA; ga.c_rpad = p->n_pad;
    first_gemm_fills = gemm_tc_supported(p, gw) && gemm_tc_supported(p, ga);
  }
  if (!first_gemm_fills) FBL_CUDA(cudaMemsetAsync(status, 0, p->zero_bytes, st));
  FBL_PROF_BEGIN();
  bool dvec_ready = false, dwo_round = false;
  {
    GemmArgs gs[2];
    GemmArgs& gw = gs[0];   // dWo = A^T dY : token-axis reduction (longest reduction loop: first in the work list)
    gw = GemmArgs{};
    gw.m = p->dq; gw.n = D; gw.n_terms = 1;
    gw.t[0] = {A, p->n_pad, 1, dY, p->n_pad, 0, n};
    gw.c = dWo; gw.c_rpad = p->dq;
    GemmArgs& ga = gs[1];   // dA = dY Wo^T : Wo's tiles read with the roles of its two axes swapped
    ga = GemmArgs{};
    ga.m = n; ga.n = p->dq; ga.n_terms = 1;
    ga.t[0] = {dY, p->n_pad, 0, Wo, p->dq, 1, D};
    ga.b_static = 1;
    ga.c = dA; ga.c_rpad = p->n_pad; ga.seq = p->d.seq; ga.t_pad = p->t_pad;
    if (p->use_tc && gemm_tc_supported(p, gw) && gemm_tc_supported(p, ga)) {
      // D = rowsum(dO * O) per head comes out of the dA epilogue, from the fp32 accumulator
      ga.dot_with = A; ga.dot_out = dvec; ga.dot_hd = p->d.head_dim; ga.dot_hq = p->d.n_q_heads;
      dvec_ready = true;
      if (split_o) { gw.ksplit = p->ksplit_o; gw.acc = (float*)(sc + p->sb_acc_o); }
      if (first_gemm_fills) {
        gs[0].zero_ptr = dqacc; gs[0].zero_bytes = p->zero_bytes - p->sb_dqacc;
        gs[0].reset_status = 1; gs[0].serial = 1;
      }
      FBL_STEP("dWo+dA", 1, launch_gemm_tc_group(p, gs, 2, status, st, FBL_GEMM_DWO_DA));
      dwo_round = split_o;        // nothing in the step reads dWo: its rounding joins that of dWq, dWk, dWv below
    } else {
      FBL_STEP("dA", 1, run_gemm(p, ga, status, st));
      FBL_STEP("dWo", 1, run_gemm(p, gw, status, st));
    }
  }
  if (p->use_tc && attn_bwd_tc_supported(p)) FBL_STEP("attn_bwd", dvec_ready ? 2 : 3, launch_attn_bwd_tc(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, dvec_ready, status, st));   // dqacc: zero already
  else FBL_STEP("attn_bwd", 3, launch_attn_bwd_simt(p, Q, K, V, A, dA, lse, dvec, dqacc, dQ, dK, dV, st));
  // back through the rotation of Q and K: its transpose is the rotation by the opposite angle
  if (p->rope_base > 0.f) FBL_STEP("rope_bwd", 1, launch_rope(p, dQ, p->d.n_q_heads, dK, p->d.n_kv_heads, 1, st));
  {
    const void* G[3] = {dQ, dK, dV};
    void* DW[3] = {dWq, dWk, dWv};
    const int cols[3] = {p->dq, p->dkv, p->dkv};
    GemmArgs gs[4];
    bool tc = p->use_tc != 0;
    for (int i = 0; i < 3; ++i) {   // dW* = Xn^T d* : token-axis reductions, Xn's tiles read MN-major
      GemmArgs& g = gs[i];
      g = GemmArgs{};
      g.m = D; g.n = cols[i]; g.n_terms = 1;
      g.t[0] = {Xn, p->n_pad, 1, G[i], p->n_pad, 0, n};
      g.c = DW[i]; g.c_rpad = D;
      tc = tc && gemm_tc_supported(p, g);
    }
    GemmArgs& gx = gs[3];           // dXn = dQ Wq^T + dK Wk^T + dV Wv^T : one accumulator, three reduction loops
    gx = GemmArgs{};
    gx.m = n; gx.n = D; gx.n_terms = 3;
    gx.t[0] = {dQ, p->n_pad, 0, Wq, D, 1, p->dq};
    gx.b_static = 1;
    gx.t[1] = {dK, p->n_pad, 0, Wk, D, 1, p->dkv};
    gx.t[2] = {dV, p->n_pad, 0, Wv, D, 1, p->dkv};
    gx.c = dXn; gx.c_rpad = p->n_pad; gx.seq = p->d.seq; gx.t_pad = p->t_pad;
    tc = tc && gemm_tc_supported(p, gx);
    if (tc) {
      ConvertGroup cg = {};
      if (split_qkv) {
        float* acc = (float*)(sc + p->sb_acc_qkv);
        for (int i = 0; i < 3; ++i) {
          gs[i].ksplit = p->ksplit_qkv; gs[i].acc = acc;
          cg.src[i] = acc; cg.dst[i] = DW[i]; cg.n[i] = up8(D) * (int64_t)cols[i];
          acc += cg.n[i];
        }
        cg.count = 3;
      }
      if (dwo_round) {
        cg.src[cg.count] = (const float*)(sc + p->sb_acc_o); cg.dst[cg.count] = dWo; cg.n[cg.count] = up8(p->dq) * (int64_t)D;
        cg.count++;
        dwo_round = false;
      }
      FBL_STEP("dWqkv+dXn", 1, launch_gemm_tc_group(p, gs, 4, status, st, FBL_GEMM_DWQKV_DXN));
      if (cg.count > 0) FBL_STEP("dW round", 1, launch_convert_f32_group(cg, st));     // one rounding launch for all sliced GEMMs
    } else {
      FBL_STEP("dXn", 1, run_gemm(p, gx, status, st));
      for (int i = 0; i < 3; ++i)
        FBL_STEP(i == 0 ? "dWq" : i == 1 ? "dWk" : "dWv", 1, run_gemm(p, gs[i], status, st));
    }
  }
  if (dwo_round) {
    ConvertGroup cg = {};
    cg.src[0] = (const float*)(sc + p->sb_acc_o); cg.dst[0] = dWo; cg.n[0] = up8(p->dq) * (int64_t)D; cg.count = 1;
    FBL_STEP("dW round", 1, launch_convert_f32_group(cg, st));
  }
  // every bias gradient is a token-axis column sum: the four of them share their launches, and the second stage
  // shares the norm backward's second kernel where that kernel exists
  const void* M4[4] = {dY, dQ, dK, dV};
  float* O4[4] = {dbo, dbq, dbk, dbv};
  const int C4[4] = {D, p->dq, p->dkv, p->dkv};
  if (bias && norm_bwd_takes_colsums(p)) {
    FBL_STEP("db+norm_bwd", 2, launch_norm_bwd(p, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, (float*)part, st, 4, M4, C4, O4));
    return FBL_OK;
  }
  if (bias) FBL_STEP("db", 2, launch_colsum_group(p->d.dtype, 4, M4, p->n_pad, C4, O4, (float*)part, st));
  FBL_STEP("norm_bwd", norm_bwd_takes_colsums(p) ? 2 : 1, launch_norm_bwd(p, dXn, X, p->d.residual ? dY : nullptr, stats, gamma, dX, dgamma, dbeta, (float*)part, st));
  return FBL_OK;
}

int fbl_colsum_scratch_bytes(const fbl_plan* plan, int64_t rows, int64_t cols, size_t* bytes) {
  if (!plan || !bytes || rows <= 0 || cols <= 0 || rows % 8 != 0 || cols % plan->tw != 0) return FBL_ERR_INVALID_ARG;
  *bytes = colsum_scratch_bytes(rows, cols);
  return FBL_OK;
}

int fbl_colsum(const fbl_plan* plan, const void* M_dev, int64_t rows, int64_t cols, float* out_dev, void* scratch_dev,
               void* stream) {
  if (!plan || !M_dev || !out_dev || !scratch_dev || rows <= 0 || cols <= 0 || rows % 8 != 0 || cols % plan->tw != 0)
    return FBL_ERR_INVALID_ARG;
  if (misaligned(M_dev)) return FBL_ERR_MISALIGNED;
  FBL_CUDA(launch_colsum(plan->d.dtype, M_dev, rows, cols, out_dev, (float*)scratch_dev, as_stream(stream)));
  return FBL_OK;
}

int fbl_status_poll(const fbl_plan* plan, const void* scratch, int32_t* device_status) {
  if (!plan || !scratch || !device_status) return FBL_ERR_INVALID_ARG;
  FBL_CUDA(cudaMemcpy(device_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToHost));
  return *device_status == 0 ? FBL_OK : FBL_ERR_TIMEOUT;
}

int fbl_selftest_wait_timeout(void* scratch, int64_t limit_cycles, void* stream) {
  if (!scratch || misaligned(scratch)) return scratch ? FBL_ERR_MISALIGNED : FBL_ERR_INVALID_ARG;
  if (limit_cycles < 1000) limit_cycles = 1000;
  if (limit_cycles > 2000000000LL) limit_cycles = 2000000000LL;
  cudaStream_t st = as_stream(stream);
  FBL_CUDA(cudaMemsetAsync(scratch, 0, 8, st));
  FBL_CUDA(launch_wait_timeout_selftest((int32_t*)scratch, (long long)limit_cycles, st));
  return FBL_OK;
}

const char* fbl_strerror(int status) {
  switch (status) {
    case FBL_OK: return "ok";
    case FBL_ERR_INVALID_ARG: return "invalid argument";
    case FBL_ERR_UNSUPPORTED_SHAPE: return "shape not supported by the tiled layout or the kernels";
    case FBL_ERR_MISALIGNED: return "matrix pointer is not 1024-byte aligned";
    case FBL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case FBL_ERR_CUDA: return "CUDA runtime error";
    case FBL_ERR_TIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
  }
}

}  // extern "C"
