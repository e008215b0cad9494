// Projection GEMMs on tcgen05 tensor cores (bf16 in, fp32 accumulate in TMEM, bf16 out), operands in
// R-Tile order fetched by TMA.  One kernel serves all six projection steps and their transposed forms:
// each operand is declared K-major or MN-major in the descriptors, so W / W^T and X / X^T are the same
// tiles in HBM and in shared memory.  Up to three reduction loops feed one accumulator (dXn), and up
// to four problems share one persistent launch (Q/K/V projections; dWo with dA; dWq/dWk/dWv with dXn).
#include <string.h>

#include <mutex>

#include "fbl_internal.h"
#include "pdl.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BK = 64;
constexpr int MAX_TERMS = 3, MAX_PROBLEMS = 4;

struct alignas(64) TcProblem {
  CUtensorMap ta[MAX_TERMS], tb[MAX_TERMS], tc;     // tc: the output, for the epilogue's bulk stores
  int n_terms;
  int b_static;                                        // 1: the first term's B operand is an input of the whole
                                                       // step (a weight), not written by an earlier kernel
  int kblocks[MAX_TERMS];
  int a_mn[MAX_TERMS], b_mn[MAX_TERMS];   // 1: operand is MN-major in shared memory (its rows are K indices)
  int m, n;
  __nv_bfloat16* c;
  long long c_rpad;
  const float* bias;
  const __nv_bfloat16* residual;
  int seq, t_pad;
  const __nv_bfloat16* dot_with;   // fused D = rowsum(C * dot_with) per head (the attention backward's D), or nullptr
  float* dot_out;
  int dot_hd, dot_hq;
};
struct alignas(64) TcGroup {
  TcProblem p[MAX_PROBLEMS];
  int count;
  int32_t* status;
};

template <int BN, int STAGES>
struct SmemPlan {
  static constexpr uint32_t A_BYTES = BM * 128;
  static constexpr uint32_t B_BYTES = BN * 128;
  static constexpr uint32_t STAGE = A_BYTES + B_BYTES;
  static constexpr uint32_t STG_OFF = STAGES * STAGE;    // two 128 x 64 bf16 output staging tiles
  static constexpr uint32_t BAR_OFF = STG_OFF + 2 * 16384;
  static constexpr uint32_t N_BARS = 2 * STAGES + 8;     // full[], empty[], acc_full[2], acc_empty[2], stg_full[2], stg_free[2]
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16 + 1024;   // + TMEM slot + alignment slack
};

// Work list of a launch: output tiles of all problems, numbered problem by problem with the M tile index
// fastest (blocks that run together then share the B tiles of one weight column block through L2).
struct TileCoord { int prob, m0, n0; };

template <int BN>
__device__ __forceinline__ bool tile_at(const TcGroup& G, int w, TileCoord* tc_out) {
  for (int p = 0; p < G.count; ++p) {
    const int tm = (G.p[p].m + BM - 1) / BM, tn = (G.p[p].n + BN - 1) / BN;
    if (w < tm * tn) {
      tc_out->prob = p;
      tc_out->m0 = (w % tm) * BM;
      tc_out->n0 = (w / tm) * BN;
      return true;
    }
    w -= tm * tn;
  }
  return false;
}

// Persistent kernel: one block per SM walks the work list with stride gridDim.x.  Warp 0 feeds the
// shared-memory ring by TMA, warp 1 issues the MMAs into one of two TMEM accumulators, warps 2-5 drain the
// other accumulator (bias, residual, padding-row mask, bf16 rows in R-Tile order), so the epilogue of
// one tile overlaps the main loop of the next.
template <int BN, int STAGES>
__global__ void __launch_bounds__(192, 1) gemm_tc_kernel(const __grid_constant__ TcGroup G) {
  using SP = SmemPlan<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + SP::BAR_OFF;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto acc_empty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  auto stg_full = [&](int a) { return bars + 8u * (2 * STAGES + 4 + a); };
  auto stg_free = [&](int a) { return bars + 8u * (2 * STAGES + 6 + a); };
  const uint32_t slot = bars + 8 * SP::N_BARS;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  int32_t* status = G.status;
  constexpr uint32_t TMEM_COLS = 2 * BN;                 // two fp32 accumulators of BN columns

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      tc::mbar_init(full(s), 1);                 // one producer arrival + transaction bytes
      tc::mbar_init(empty(s), 1);                // one tcgen05.commit arrival
    }
    for (int a = 0; a < 2; ++a) {
      tc::mbar_init(acc_full(a), 1);
      tc::mbar_init(acc_empty(a), 128);
      tc::mbar_init(stg_full(a), 128);
      tc::mbar_init(stg_free(a), 1);
    }
    tc::fence_barrier_init();
  }
  if (warp == 1) {
    tc::tmem_alloc(slot, TMEM_COLS);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(slot));
  pdl_launch_dependents();

  if (warp == 0 && lane == 0) {
    // ---- TMA producer ----------------------------------------------------------------------
    int it = 0;
    bool ok = true;
    TileCoord tcd;
    // Weights do not depend on the kernel before this one: their tiles for the first stages of the first
    // output tile are requested before waiting for that kernel, hiding their (cold) latency.
    int prefilled = 0;
    if (tile_at<BN>(G, blockIdx.x, &tcd) && G.p[tcd.prob].b_static) {
      const TcProblem& P = G.p[tcd.prob];
      tc::tma_prefetch_desc(&P.ta[0]);
      tc::tma_prefetch_desc(&P.tb[0]);
      const int n = P.kblocks[0] < STAGES ? P.kblocks[0] : STAGES;
      for (int kb = 0; kb < n; ++kb) {
        const uint32_t sb = base + kb * SP::STAGE + SP::A_BYTES;
        tc::mbar_expect_tx(full(kb), SP::STAGE);
        if (P.b_mn[0]) tc::tma_load_3d(sb, &P.tb[0], full(kb), 0, kb * BK, tcd.n0 / 64);
        else tc::tma_load_3d(sb, &P.tb[0], full(kb), 0, tcd.n0, kb);
      }
      prefilled = n;
    }
    pdl_wait();
    for (int w = blockIdx.x; ok && tile_at<BN>(G, w, &tcd); w += gridDim.x) {
      const TcProblem& P = G.p[tcd.prob];
      for (int t = 0; t < P.n_terms && ok; ++t) {
        for (int kb = 0; kb < P.kblocks[t]; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          const uint32_t sa = base + s * SP::STAGE, sb = sa + SP::A_BYTES;
          const bool pre = it < prefilled;                 // this stage's barrier is armed and its B tile on its way
          if (!pre) {
            if (!tc::mbar_wait(empty(s), ph ^ 1, status, 101)) { ok = false; break; }
            tc::mbar_expect_tx(full(s), SP::STAGE);
          }
          if (P.a_mn[t]) tc::tma_load_3d(sa, &P.ta[t], full(s), 0, kb * BK, tcd.m0 / 64);
          else tc::tma_load_3d(sa, &P.ta[t], full(s), 0, tcd.m0, kb);
          if (!pre) {
            if (P.b_mn[t]) tc::tma_load_3d(sb, &P.tb[t], full(s), 0, kb * BK, tcd.n0 / 64);
            else tc::tma_load_3d(sb, &P.tb[t], full(s), 0, tcd.n0, kb);
          }
        }
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer ------------------------------------------------------------------------
    int it = 0, ti = 0;
    bool ok = true;
    TileCoord tcd;
    for (int w = blockIdx.x; ok && tile_at<BN>(G, w, &tcd); w += gridDim.x, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      if (!tc::mbar_wait(acc_empty(ab), ((ti >> 1) & 1) ^ 1, status, 104)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t d_tmem = tmem_base + ab * BN;
      bool first = true;
      for (int t = 0; t < P.n_terms && ok; ++t) {
        const uint32_t idesc = tc::idesc_bf16(BM, BN, P.a_mn[t], P.b_mn[t]);
        // K-major: 8-row groups 1024 B apart, 16 K elements = 32 B along the row.
        // MN-major: 64-wide M/N blocks 8 KiB apart (64 K rows x 128 B), 16 K rows = 2 KiB.
        const uint32_t a_lbo = P.a_mn[t] ? 8192u : 16u, a_step = P.a_mn[t] ? 2048u : 32u;
        const uint32_t b_lbo = P.b_mn[t] ? 8192u : 16u, b_step = P.b_mn[t] ? 2048u : 32u;
        for (int kb = 0; kb < P.kblocks[t]; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!tc::mbar_wait(full(s), ph, status, 102)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t sa = base + s * SP::STAGE, sb = sa + SP::A_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            const uint64_t da = tc::smem_desc_sw128(sa + kk * a_step, a_lbo, 1024);
            const uint64_t db = tc::smem_desc_sw128(sb + kk * b_step, b_lbo, 1024);
            tc::mma_bf16_ss(d_tmem, da, db, idesc, (first && kk == 0) ? 0u : 1u);
          }
          first = false;
          tc::mma_commit(empty(s));              // frees the stage once these MMAs have read it
        }
      }
      if (ok) tc::mma_commit(acc_full(ab));
    }
  } else if (warp >= 2) {
    // ---- epilogue: TMEM -> registers -> swizzled staging tile -> bulk tensor store, one 64-column panel at
    // a time (two staging tiles: the store of one panel overlaps the conversion of the next) -------------
    pdl_wait();                                       // the previous kernel may still be reading what we overwrite
    const int q = warp % 4;                           // the TMEM lane quarter this warp may access
    const int r = q * 32 + lane;                      // row of the tile owned by this thread
    const bool issuer = threadIdx.x == 64;
    int ti = 0, pc = 0;                               // tiles and panels done by this block
    bool ok = true;
    TileCoord tcd;
    for (int w = blockIdx.x; ok && tile_at<BN>(G, w, &tcd); w += gridDim.x, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      if (!tc::mbar_wait(acc_full(ab), (ti >> 1) & 1, status, 103)) { ok = false; break; }
      tc::tc_fence_after();
      const int row = tcd.m0 + r;
      const bool pad = P.t_pad > 0 && (row % P.t_pad) >= P.seq;
      float dot_acc = 0.f;
#pragma unroll 1
      for (int pn = 0; pn < BN / 64 && ok; ++pn) {
        const int n = tcd.n0 + pn * 64;
        if (n >= P.n) break;                           // uniform: N is whole 64-column panels
        uint32_t v[64];
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
        tc::tmem_ld_wait();
        uint4 outv[8];
        uint32_t* ow = reinterpret_cast<uint32_t*>(outv);
        if (P.residual && row < P.m) {
          const __nv_bfloat16* rp = P.residual + ((long long)(n / 64) * P.c_rpad + row) * 64;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 rv = *reinterpret_cast<const uint4*>(rp + 8 * j);
            const __nv_bfloat16* rb = reinterpret_cast<const __nv_bfloat16*>(&rv);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[8 * j + k] = __float_as_uint(__uint_as_float(v[8 * j + k]) + __bfloat162float(rb[k]));
          }
        }
#pragma unroll
        for (int j = 0; j < 64; j += 2) {
          float v0 = __uint_as_float(v[j]), v1 = __uint_as_float(v[j + 1]);
          if (P.bias) { v0 += P.bias[n + j]; v1 += P.bias[n + j + 1]; }
          if (pad) { v0 = 0.f; v1 = 0.f; }
          ow[j / 2] = tc::pack_bf16(v0, v1);
        }
        if (P.dot_with && row < P.m) {
          // Row reduction over this head's columns, on the ROUNDED values the attention backward will read:
          // sum_j dS_ij = 0 (softmax shift invariance) holds only if D matches the dP that kernel forms.
          const __nv_bfloat16* ap = P.dot_with + ((long long)(n / 64) * P.c_rpad + row) * 64;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 av = *reinterpret_cast<const uint4*>(ap + 8 * j);
            const __nv_bfloat16* ab16 = reinterpret_cast<const __nv_bfloat16*>(&av);
#pragma unroll
            for (int k = 0; k < 8; k += 2) {
              const uint32_t w2 = ow[4 * j + k / 2];        // two bf16: low half = even column
              dot_acc = fmaf(__uint_as_float(w2 << 16), __bfloat162float(ab16[k]), dot_acc);
              dot_acc = fmaf(__uint_as_float(w2 & 0xffff0000u), __bfloat162float(ab16[k + 1]), dot_acc);
            }
          }
          if ((n + 64) % P.dot_hd == 0) {                 // last panel of a head
            const int hh = n / P.dot_hd, bb = row / P.t_pad, tt = row % P.t_pad;
            P.dot_out[((long long)bb * P.dot_hq + hh) * P.t_pad + tt] = dot_acc;
            dot_acc = 0.f;
          }
        }
        const int sb = pc & 1;
        const uint32_t stg = base + SP::STG_OFF + sb * 16384;
        // the staging tile's previous store (two panels ago) must have read it
        if (pc >= 2 && !tc::mbar_wait(stg_free(sb), ((pc >> 1) - 1) & 1, status, 105)) { ok = false; break; }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + r * 128 + (((uint32_t)j ^ (uint32_t)(r & 7)) * 16)),
                       "r"(outv[j].x), "r"(outv[j].y), "r"(outv[j].z), "r"(outv[j].w) : "memory");
        tc::fence_proxy_async();
        tc::mbar_arrive(stg_full(sb));
        if (issuer) {
          if (!tc::mbar_wait(stg_full(sb), (pc >> 1) & 1, status, 106)) { ok = false; break; }
          tc::tma_store_3d(&P.tc, stg, 0, tcd.m0, n / 64);
          tc::bulk_commit_group();
          if (pc >= 1) {                               // at most this store in flight: the previous one has read
            tc::bulk_wait_group_read1();               // its staging tile, which may now be overwritten
            tc::mbar_arrive(stg_free(sb ^ 1));
          }
        }
        ++pc;
      }
      tc::tc_fence_before();
      tc::mbar_arrive(acc_empty(ab));             // this accumulator may be overwritten by the tile after next
    }
    if (issuer) tc::bulk_wait_group0();           // all output tiles are in global memory before the block exits
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

constexpr int BN_SMALL = 128;

}  // namespace

bool fbl_encode_rtile_map(CUtensorMap* map, const void* base, int64_t r_pad, int panels, int box_rows, int box_panels) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {64, (cuuint64_t)r_pad, (cuuint64_t)panels};
  cuuint64_t strides[2] = {128, (cuuint64_t)r_pad * 128};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_panels};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 accumulator [n_pad, cols] stored in the bf16 tile order (64-column panels, 256-byte rows), viewed as
// [panels][rows][2 halves][32 floats] so that a box of 128 rows x one panel can use the 128-byte swizzle.
bool fbl_encode_f32_panel_map(CUtensorMap* map, const void* base, int64_t r_pad, int panels, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {32, 2, (cuuint64_t)r_pad, (cuuint64_t)panels};
  cuuint64_t strides[3] = {128, 256, (cuuint64_t)r_pad * 256};
  cuuint32_t box[4] = {32, 2, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_tc_supported(const fbl_plan* p, const GemmArgs& g) {
  if (p->d.dtype != FBL_DTYPE_BF16) return false;
  if (g.n % 64 != 0 || g.n < BN_SMALL || g.m < BM) return false;
  for (int t = 0; t < g.n_terms; ++t) {
    const GemmTerm& tm = g.t[t];
    // a box must fit inside its tensor: rows of every operand cover one tile, K-major reduction axes are whole panels
    if (tm.a_trans ? (tm.k < BK || g.m % 64 != 0) : (tm.k % BK != 0)) return false;
    if (tm.b_trans ? (tm.k % BK != 0) : (tm.k < BK)) return false;
    if (tm.a_rpad < 128 || tm.b_rpad < 128) return false;
  }
  return true;
}

template <int BN, int STAGES>
cudaError_t launch_group_bn(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st) {
  TcGroup G;
  memset(&G, 0, sizeof(G));
  G.count = count;
  G.status = status;
  int tiles = 0;
  for (int i = 0; i < count; ++i) {
    const GemmArgs& g = gs[i];
    TcProblem& P = G.p[i];
    P.n_terms = g.n_terms;
    for (int t = 0; t < g.n_terms; ++t) {
      const GemmTerm& tm = g.t[t];
      P.kblocks[t] = (tm.k + BK - 1) / BK;
      P.a_mn[t] = tm.a_trans ? 1 : 0;     // stored [k rows][m cols]: rows are K indices
      P.b_mn[t] = tm.b_trans ? 0 : 1;     // stored [k rows][n cols]: rows are K indices
      bool ok;
      if (tm.a_trans) ok = fbl_encode_rtile_map(&P.ta[t], tm.a, tm.a_rpad, g.m / 64, BK, BM / 64);
      else ok = fbl_encode_rtile_map(&P.ta[t], tm.a, tm.a_rpad, tm.k / 64, BM, 1);
      if (!ok) return cudaErrorInvalidValue;
      if (tm.b_trans) ok = fbl_encode_rtile_map(&P.tb[t], tm.b, tm.b_rpad, tm.k / 64, BN, 1);
      else ok = fbl_encode_rtile_map(&P.tb[t], tm.b, tm.b_rpad, g.n / 64, BK, BN / 64);
      if (!ok) return cudaErrorInvalidValue;
    }
    P.m = g.m; P.n = g.n;
    if (!fbl_encode_rtile_map(&P.tc, g.c, g.c_rpad, g.n / 64, BM, 1)) return cudaErrorInvalidValue;
    P.b_static = g.b_static;
    P.c = (__nv_bfloat16*)g.c; P.c_rpad = g.c_rpad;
    P.bias = g.bias; P.residual = (const __nv_bfloat16*)g.residual;
    P.seq = g.seq; P.t_pad = g.t_pad;
    P.dot_with = (const __nv_bfloat16*)g.dot_with; P.dot_out = g.dot_out; P.dot_hd = g.dot_hd; P.dot_hq = g.dot_hq;
    tiles += ((g.m + BM - 1) / BM) * ((g.n + BN - 1) / BN);
  }
  using SP = SmemPlan<BN, STAGES>;
  auto k = gemm_tc_kernel<BN, STAGES>;
  cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
  if (attr_err != cudaSuccess) return attr_err;
  const int grid = tiles < p->sm_count ? tiles : p->sm_count;
  return launch_pdl(k, dim3(grid), dim3(192), SP::TOTAL, st, G);
}

cudaError_t launch_gemm_tc_group(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st) {
  if (count < 1 || count > MAX_PROBLEMS) return cudaErrorInvalidValue;
  bool wide = true;                       // 128 x 256 tiles when every problem's N is whole 256-column blocks
  int tiles_wide = 0;
  for (int i = 0; i < count; ++i) {
    wide = wide && gs[i].n % 256 == 0;
    for (int t = 0; t < gs[i].n_terms; ++t)
      if (gs[i].t[t].b_trans && gs[i].t[t].b_rpad < 256) wide = false;
    tiles_wide += ((gs[i].m + BM - 1) / BM) * ((gs[i].n + 255) / 256);
  }
  // with too few wide tiles to occupy the SMs, narrower tiles (twice as many) finish sooner
  if (wide && tiles_wide * 3 < p->sm_count * 2) wide = false;
  if (wide) return launch_group_bn<256, 4>(p, gs, count, status, st);
  return launch_group_bn<128, 6>(p, gs, count, status, st);
}

cudaError_t launch_gemm_tc(const fbl_plan* p, const GemmArgs& g, void*, size_t, int32_t* status, cudaStream_t st) {
  return launch_gemm_tc_group(p, &g, 1, status, st);
}
