// Projection GEMMs on tcgen05 tensor cores (bf16 in, fp32 accumulate in TMEM, bf16 out), operands in
// R-Tile order fetched by TMA.  One kernel serves all six projection steps and their transposed forms:
// each operand is declared K-major or MN-major in the descriptors, so W / W^T and X / X^T are the same
// tiles in HBM and in shared memory.  Up to three reduction loops feed one accumulator (dXn), and up
// to four problems share one persistent launch (Q/K/V projections; dWo with dA; dWq/dWk/dWv with dXn).
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "fbl_internal.h"
#include "pdl.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BK = 64;
constexpr int MAX_TERMS = 4, MAX_PROBLEMS = 5;

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
  // Reduction loop cut into `ksplit` slices, each a work unit of its own (a problem with few output tiles and a
  // long reduction): slices add their fp32 partial tiles into `tacc`'s buffer with bulk tensor reductions, and a
  // later kernel rounds the sums to bf16.  Single-term problems without epilogue extras only.
  int ksplit;
  CUtensorMap tacc;
  // Fused activation of the feed-forward block (kernel variant EPI only; `residual` then points at the first extra
  // operand U instead of a residual, `aux1` at the second one, G; `tc2` is the second output's map):
  //   1 GELU forward    C = v (U), C2 = gelu(v)           2 GELU backward    C = v gelu'(U)
  //   3 gated forward   C = v (G), C2 = silu(v) U          4 gated backward   C = v silu(G), C2 = v U silu'(G)
  int epi;
  const __nv_bfloat16* aux1;
  CUtensorMap tc2;
};
struct alignas(64) TcGroup {
  TcProblem p[MAX_PROBLEMS];
  int count;
  int32_t* status;
  // Optional chores for the epilogue warps while the first tile's main loop runs: zero-fill a buffer that a later
  // kernel of the pass adds into (16-byte units, dealt evenly to the blocks), and reset the pass's status word.
  uint4* zero_ptr;
  long long zero_vec;
  int reset_status;
};

__device__ __forceinline__ void group_chores(const TcGroup& G, int tid, int n_threads) {
  if (G.reset_status && blockIdx.x == 0 && tid == 0) *G.status = 0;
  if (G.zero_vec > 0) {
    const long long per = (G.zero_vec + gridDim.x - 1) / gridDim.x;
    const long long lo = (long long)blockIdx.x * per, hi = min(G.zero_vec, lo + per);
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (long long i = lo + tid; i < hi; i += n_threads) G.zero_ptr[i] = z;
  }
}

template <int BN, int STAGES>
struct SmemPlan {
  static constexpr uint32_t A_BYTES = BM * 128;
  static constexpr uint32_t B_BYTES = BN * 128;
  static constexpr uint32_t STAGE = A_BYTES + B_BYTES;
  static constexpr uint32_t STG_OFF = STAGES * STAGE;    // per epilogue warp two 32 x 64 bf16 output staging tiles
  static constexpr uint32_t BAR_OFF = STG_OFF + 2 * 16384;
  static constexpr uint32_t N_BARS = 2 * STAGES + 4;     // full[], empty[], acc_full[2], acc_empty[2]
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16 + 1024;   // + TMEM slot + alignment slack
};

// Work list of a launch: output tiles of all problems, numbered problem by problem with the M tile index
// fastest (blocks that run together then share the B tiles of one weight column block through L2).
struct TileCoord { int prob, m0, n0, kb0, kb1; };     // kb0..kb1: k-block range of term 0 (split problems)

template <int BN>
__device__ __forceinline__ bool tile_at(const TcGroup& G, int w, TileCoord* tc_out) {
  for (int p = 0; p < G.count; ++p) {
    const TcProblem& P = G.p[p];
    const int tm = (P.m + BM - 1) / BM, tn = (P.n + BN - 1) / BN;
    const int units = tm * tn * P.ksplit;
    if (w < units) {
      const int slice = w % P.ksplit, t = w / P.ksplit;        // slices of one tile are neighbours in the list
      tc_out->prob = p;
      tc_out->m0 = (t % tm) * BM;
      tc_out->n0 = (t / tm) * BN;
      const int per = (P.kblocks[0] + P.ksplit - 1) / P.ksplit;
      tc_out->kb0 = slice * per;
      tc_out->kb1 = min(P.kblocks[0], (slice + 1) * per);
      return true;
    }
    w -= units;
  }
  return false;
}

// Persistent kernel: one block per SM walks the work list with stride gridDim.x.  Warp 0 feeds the
// shared-memory ring by TMA, warp 1 issues the MMAs into one of two TMEM accumulators, warps 2-5 drain the
// other accumulator (bias, residual, padding-row mask, bf16 rows in R-Tile order), so the epilogue of
// one tile overlaps the main loop of the next.
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float gelu_fast(float u) { return 0.5f * u * (1.f + tanh_fast(0.7978845608028654f * (u + 0.044715f * u * u * u))); }
__device__ __forceinline__ float gelu_grad_fast(float u) {
  const float t = tanh_fast(0.7978845608028654f * (u + 0.044715f * u * u * u));
  return 0.5f * (1.f + t) + 0.5f * u * (1.f - t * t) * 0.7978845608028654f * (1.f + 0.134145f * u * u);
}
__device__ __forceinline__ float sigmoid_fast(float g) { return __fdividef(1.f, 1.f + __expf(-g)); }

template <int BN, int STAGES, int ESETS, bool EPI = false>
__global__ void __launch_bounds__(64 + 128 * ESETS, 1) gemm_tc_kernel(const __grid_constant__ TcGroup G) {
  using SP = SmemPlan<BN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + SP::BAR_OFF;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto acc_empty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
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
      tc::mbar_init(acc_empty(a), 128 * ESETS);
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
    if (tile_at<BN>(G, blockIdx.x, &tcd) && G.p[tcd.prob].b_static && G.p[tcd.prob].ksplit == 1) {
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
        const int kb_begin = t == 0 ? tcd.kb0 : 0, kb_end = t == 0 ? tcd.kb1 : P.kblocks[t];
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
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
    // ---- MMA issuer: one thread.  Descriptor words are formed once per reduction loop; per instruction only
    // the start-address field moves.  (The loop is not the limit: with 128 x 256 tiles a k-block's 48 KB of
    // operands take longer to arrive from L2, at about 64 B/clk per SM, than its four MMAs take to run.) ------
    int s = 0, ti = 0;
    uint32_t ph = 0;
    bool ok = true;
    TileCoord tcd;
    const uint32_t hi = tc::smem_desc_hi(1024);
    for (int w = blockIdx.x; ok && tile_at<BN>(G, w, &tcd); w += gridDim.x, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      if (!tc::mbar_wait(acc_empty(ab), ((ti >> 1) & 1) ^ 1, status, 104)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t d_tmem = tmem_base + ab * BN;
      uint32_t acc = 0;
      for (int t = 0; t < P.n_terms && ok; ++t) {
        const uint32_t idesc = tc::idesc_bf16(BM, BN, P.a_mn[t], P.b_mn[t]);
        // K-major: 8-row groups 1024 B apart, 16 K elements = 32 B along the row.
        // MN-major: 64-wide M/N blocks 8 KiB apart (64 K rows x 128 B), 16 K rows = 2 KiB.
        const uint32_t a_lo0 = tc::smem_desc_lo(base, P.a_mn[t] ? 8192u : 16u), a_step = P.a_mn[t] ? 128u : 2u;
        const uint32_t b_lo0 = tc::smem_desc_lo(base + SP::A_BYTES, P.b_mn[t] ? 8192u : 16u), b_step = P.b_mn[t] ? 128u : 2u;
        const int nkb = t == 0 ? tcd.kb1 - tcd.kb0 : P.kblocks[t];
        for (int kb = 0; kb < nkb; ++kb) {
          if (!tc::mbar_wait(full(s), ph, status, 102)) { ok = false; break; }
          tc::tc_fence_after();
          uint32_t a_lo = a_lo0 + (uint32_t)s * (SP::STAGE >> 4), b_lo = b_lo0 + (uint32_t)s * (SP::STAGE >> 4);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            tc::mma_bf16_ss_w(d_tmem, a_lo, hi, b_lo, hi, idesc, acc);
            acc = 1;
            a_lo += a_step; b_lo += b_step;
          }
          tc::mma_commit(empty(s));              // frees the stage once these MMAs have read it
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
      if (ok) tc::mma_commit(acc_full(ab));
    }
  } else if (warp >= 2) {
    // ---- epilogue: TMEM -> registers -> swizzled staging -> bulk tensor store.  Each warp owns the 32 rows of
    // its TMEM lane quarter and two 32 x 64 staging tiles, and issues its own stores: no block-wide hand-off per
    // panel, and the store of one panel overlaps the conversion of the next. ---------------------------------
    pdl_wait();                                       // the previous kernel may still be reading what we overwrite
    group_chores(G, threadIdx.x - 64, 128 * ESETS);
    const int q = warp % 4;                           // the TMEM lane quarter this warp may access
    // ESETS = 2 (launches in which every block has a single tile, so that nothing overlaps its epilogue): two sets
    // of four warps share the tile's 64-column panels, first and second half, and the epilogue takes half as long.
    // Each warp then has one staging tile instead of two (the staging area is the same size).
    const int set = (warp - 2) / 4;
    constexpr int PPS = BN / 64 / ESETS;              // panels per set
    const int r = q * 32 + lane;                      // row of the tile owned by this thread
    int ti = 0, pc = 0;                               // tiles and panels done by this warp
    bool ok = true;
    TileCoord tcd;
    for (int w = blockIdx.x; ok && tile_at<BN>(G, w, &tcd); w += gridDim.x, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      const int row = tcd.m0 + r;
      const bool pad = P.t_pad > 0 && (row % P.t_pad) >= P.seq;
      const bool has_res = P.residual && row < P.m;
      // a head of the fused row reduction must stay within one warp: where it spans more panels than a set has, the
      // first set takes the whole tile
      const bool whole = ESETS == 2 && P.dot_with && P.dot_hd > 64 * PPS;
      const int pn_begin = set == 0 ? 0 : (whole ? BN / 64 : PPS);
      const int pn_end = ESETS == 1 ? BN / 64 : (set == 0 ? (whole ? BN / 64 : PPS) : BN / 64);
      uint4 rv[8];                                    // residual values of the next panel, requested a panel ahead
      if (has_res && pn_begin < pn_end && tcd.n0 + pn_begin * 64 < P.n) {
        const __nv_bfloat16* rp = P.residual + ((long long)(tcd.n0 / 64 + pn_begin) * P.c_rpad + row) * 64;
#pragma unroll
        for (int j = 0; j < 8; ++j) rv[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
      }
      uint4 rv2[EPI ? 8 : 1];                         // second extra operand of a fused activation, likewise
      if constexpr (EPI) {
        if (P.epi == 4 && row < P.m && pn_begin < pn_end && tcd.n0 + pn_begin * 64 < P.n) {
          const __nv_bfloat16* rp = P.aux1 + ((long long)(tcd.n0 / 64 + pn_begin) * P.c_rpad + row) * 64;
#pragma unroll
          for (int j = 0; j < 8; ++j) rv2[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
        }
      }
      const float* bias = P.bias;
      float bl[BN / 32];                              // this tile's bias: lane l holds columns l*BN/32 ... (requested
      if (bias) {                                     // while the MMAs run, handed out by shuffles below)
#pragma unroll
        for (int k = 0; k < BN / 32; ++k) {
          const int c = tcd.n0 + lane * (BN / 32) + k;
          bl[k] = c < P.n ? bias[c] : 0.f;
        }
      }
      if (!tc::mbar_wait(acc_full(ab), (ti >> 1) & 1, status, 103)) { ok = false; break; }
      tc::tc_fence_after();
      float dot_acc = 0.f;
#pragma unroll 1
      for (int pn = pn_begin; pn < pn_end; ++pn) {
        const int n = tcd.n0 + pn * 64;
        if (n >= P.n) break;                           // uniform: N is whole 64-column panels
        uint32_t v[64];
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
        tc::tmem_ld_wait();
        if (P.ksplit > 1) {
          // partial sums of a reduction slice: two 32-column halves of the panel, fp32, added to the accumulation
          // buffer by bulk tensor reductions (same staging tiles and swizzle as the bf16 rows below)
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) {
            const uint32_t stg = base + SP::STG_OFF + (ESETS == 2 ? (uint32_t)(warp - 2) : (uint32_t)(q * 2 + (pc & 1))) * 4096u;
            if (ESETS == 2 && lane == 0) tc::bulk_wait_group_read0();     // the single staging tile's previous contents have been read
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)j ^ (uint32_t)(lane & 7)) * 16)),
                           "r"(hf ? v[32 + 4 * j] : v[4 * j]), "r"(hf ? v[33 + 4 * j] : v[4 * j + 1]),
                           "r"(hf ? v[34 + 4 * j] : v[4 * j + 2]), "r"(hf ? v[35 + 4 * j] : v[4 * j + 3]) : "memory");
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tc::tma_reduce_add_4d(&P.tacc, stg, 0, hf, tcd.m0 + q * 32, n / 64);
              tc::bulk_commit_group();
              if (ESETS == 1) tc::bulk_wait_group_read1();
            }
            ++pc;
          }
          continue;
        }
        if constexpr (EPI) {
          if (P.epi != 0) {
            // ---- fused activation: one or two outputs from this panel ------------------------------------
            if (bias) {
#pragma unroll
              for (int j = 0; j < 64; ++j)
                v[j] = __float_as_uint(__uint_as_float(v[j]) + __shfl_sync(0xffffffffu, bl[j % (BN / 32)], (pn * 64 + j) / (BN / 32)));
            }
            uint4 o1[8], o2[8];
            uint32_t* w1 = reinterpret_cast<uint32_t*>(o1);
            uint32_t* w2 = reinterpret_cast<uint32_t*>(o2);
            const bool live = !pad && row < P.m;
            const __nv_bfloat16* a0 = reinterpret_cast<const __nv_bfloat16*>(rv);
            const __nv_bfloat16* a1 = reinterpret_cast<const __nv_bfloat16*>(rv2);
            const float keep = live ? 1.f : 0.f;            // padding rows and rows past the matrix are written as zero
            if (P.epi == 1) {
#pragma unroll
              for (int j = 0; j < 64; j += 2) {
                const float x0 = __uint_as_float(v[j]) * keep, x1 = __uint_as_float(v[j + 1]) * keep;
                w1[j / 2] = tc::pack_bf16(x0, x1);
                w2[j / 2] = tc::pack_bf16(gelu_fast(x0), gelu_fast(x1));
              }
            } else if (P.epi == 2) {
#pragma unroll
              for (int j = 0; j < 64; j += 2) {
                const float x0 = __uint_as_float(v[j]) * keep, x1 = __uint_as_float(v[j + 1]) * keep;
                w1[j / 2] = tc::pack_bf16(x0 * gelu_grad_fast(__bfloat162float(a0[j])), x1 * gelu_grad_fast(__bfloat162float(a0[j + 1])));
              }
            } else if (P.epi == 3) {
#pragma unroll
              for (int j = 0; j < 64; j += 2) {
                const float x0 = __uint_as_float(v[j]) * keep, x1 = __uint_as_float(v[j + 1]) * keep;
                w1[j / 2] = tc::pack_bf16(x0, x1);
                w2[j / 2] = tc::pack_bf16(x0 * sigmoid_fast(x0) * __bfloat162float(a0[j]), x1 * sigmoid_fast(x1) * __bfloat162float(a0[j + 1]));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 64; j += 2) {
                float y1[2], y2[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                  const float x = __uint_as_float(v[j + u]) * keep;
                  const float uu = __bfloat162float(a0[j + u]), gg = __bfloat162float(a1[j + u]), sg = sigmoid_fast(gg);
                  y1[u] = x * gg * sg;
                  y2[u] = x * uu * sg * (1.f + gg * (1.f - sg));
                }
                w1[j / 2] = tc::pack_bf16(y1[0], y1[1]);
                w2[j / 2] = tc::pack_bf16(y2[0], y2[1]);
              }
            }
            // the next panel's extra operands, requested while this panel's stores are under way
            if (pn + 1 < pn_end && n + 64 < P.n && row < P.m) {
              if (P.epi >= 2) {
                const __nv_bfloat16* rp = P.residual + ((long long)(n / 64 + 1) * P.c_rpad + row) * 64;
#pragma unroll
                for (int j = 0; j < 8; ++j) rv[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
              }
              if (P.epi == 4) {
                const __nv_bfloat16* rp = P.aux1 + ((long long)(n / 64 + 1) * P.c_rpad + row) * 64;
#pragma unroll
                for (int j = 0; j < 8; ++j) rv2[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
              }
            }
            const int n_out = (P.epi == 2) ? 1 : 2;
#pragma unroll 1
            for (int oi = 0; oi < n_out; ++oi) {
              const uint4* ov = oi ? o2 : o1;
              const uint32_t stg = base + SP::STG_OFF + (ESETS == 2 ? (uint32_t)(warp - 2) : (uint32_t)(q * 2 + (pc & 1))) * 4096u;
              if (ESETS == 2 && lane == 0) tc::bulk_wait_group_read0();
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 8; ++j)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)j ^ (uint32_t)(lane & 7)) * 16)),
                             "r"(ov[j].x), "r"(ov[j].y), "r"(ov[j].z), "r"(ov[j].w) : "memory");
              tc::fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                tc::tma_store_3d(oi ? &P.tc2 : &P.tc, stg, 0, tcd.m0 + q * 32, n / 64);
                tc::bulk_commit_group();
                if (ESETS == 1) tc::bulk_wait_group_read1();
              }
              ++pc;
            }
            continue;
          }
        }
        uint4 outv[8];
        uint32_t* ow = reinterpret_cast<uint32_t*>(outv);
        if (has_res) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const __nv_bfloat16* rb = reinterpret_cast<const __nv_bfloat16*>(&rv[j]);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[8 * j + k] = __float_as_uint(__uint_as_float(v[8 * j + k]) + __bfloat162float(rb[k]));
          }
          if (pn + 1 < pn_end && n + 64 < P.n) {
            const __nv_bfloat16* rp = P.residual + ((long long)(n / 64 + 1) * P.c_rpad + row) * 64;
#pragma unroll
            for (int j = 0; j < 8; ++j) rv[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
          }
        }
        if (bias) {
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            // column pn*64 + j is register (j % (BN/32)) of lane (pn*64 + j) / (BN/32)
            const float b0 = __shfl_sync(0xffffffffu, bl[j % (BN / 32)], (pn * 64 + j) / (BN / 32));
            const float b1 = __shfl_sync(0xffffffffu, bl[(j + 1) % (BN / 32)], (pn * 64 + j + 1) / (BN / 32));
            ow[j / 2] = tc::pack_bf16(pad ? 0.f : __uint_as_float(v[j]) + b0, pad ? 0.f : __uint_as_float(v[j + 1]) + b1);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 64; j += 2)
            ow[j / 2] = tc::pack_bf16(pad ? 0.f : __uint_as_float(v[j]), pad ? 0.f : __uint_as_float(v[j + 1]));
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
        // Staging tile (pc & 1) of this warp: its previous store (two panels ago) has been read, since lane 0
        // waited for that after committing the store of the panel before this one.
        const uint32_t stg = base + SP::STG_OFF + (ESETS == 2 ? (uint32_t)(warp - 2) : (uint32_t)(q * 2 + (pc & 1))) * 4096u;
        if (ESETS == 2 && lane == 0) tc::bulk_wait_group_read0();    // one staging tile: the store before has read it
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)j ^ (uint32_t)(lane & 7)) * 16)),
                       "r"(outv[j].x), "r"(outv[j].y), "r"(outv[j].z), "r"(outv[j].w) : "memory");
        tc::fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          tc::tma_store_3d(&P.tc, stg, 0, tcd.m0 + q * 32, n / 64);
          tc::bulk_commit_group();
          if (ESETS == 1) tc::bulk_wait_group_read1();  // the store before this one has read its staging tile
        }
        ++pc;
      }
      tc::tc_fence_before();
      tc::mbar_arrive(acc_empty(ab));             // this accumulator may be overwritten by the tile after next
    }
    if (lane == 0) tc::bulk_wait_group0();        // all output tiles are in global memory before the block exits
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------------
// CTA-pair variant (tcgen05 cta_group::2): two SMs share a 256 x 256 output tile.  Each CTA loads its 128 rows of
// A and its 128 columns of B (32 KB per k-block instead of 48 KB for a 128 x 256 tile of its own: operand
// delivery from L2, about 64 B/clk per SM, is what bounds the single-CTA kernel), the leader (cluster rank 0)
// issues MMAs of M = 256, N = 256 that read both CTAs' shared memory and write 128 accumulator rows into each
// CTA's tensor memory, and each CTA drains its own rows.  Barriers: full[] lives in the leader and counts the
// bytes of both CTAs' loads; empty[] and acc_full[] exist in both and get their arrivals from one commit that
// signals both CTAs; acc_empty[] lives in the leader and takes the arrivals of both CTAs' epilogue threads.
// ---------------------------------------------------------------------------------------------------
constexpr int PAIR_BN = 256, PAIR_STAGES = 6;
struct PairSmem {
  static constexpr uint32_t A_BYTES = 128 * 128, B_BYTES = 128 * 128, STAGE = A_BYTES + B_BYTES;
  static constexpr uint32_t STG_OFF = PAIR_STAGES * STAGE;
  static constexpr uint32_t BAR_OFF = STG_OFF + 2 * 16384;
  static constexpr uint32_t N_BARS = 2 * PAIR_STAGES + 4;
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16 + 1024;
};

// work list in 256 x 256 tiles (ksplit slices as in tile_at); m0 / n0 are the pair's
__device__ __forceinline__ bool pair_tile_at(const TcGroup& G, int w, TileCoord* tc_out) {
  for (int p = 0; p < G.count; ++p) {
    const TcProblem& P = G.p[p];
    const int tm = (P.m + 255) / 256, tn = (P.n + 255) / 256;
    const int units = tm * tn * P.ksplit;
    if (w < units) {
      const int slice = w % P.ksplit, t = w / P.ksplit;
      tc_out->prob = p;
      tc_out->m0 = (t % tm) * 256;
      tc_out->n0 = (t / tm) * 256;
      const int per = (P.kblocks[0] + P.ksplit - 1) / P.ksplit;
      tc_out->kb0 = slice * per;
      tc_out->kb1 = min(P.kblocks[0], (slice + 1) * per);
      return true;
    }
    w -= units;
  }
  return false;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 1) gemm_tc_pair_kernel(const __grid_constant__ TcGroup G) {
  using SP = PairSmem;
  constexpr int STAGES = PAIR_STAGES, BN = PAIR_BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + SP::BAR_OFF;
  auto full = [&](int s) { return bars + 8u * s; };
  auto empty = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto acc_empty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  const uint32_t slot = bars + 8 * SP::N_BARS;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const uint32_t rank = tc::cluster_ctarank();
  const int pair_id = blockIdx.x / 2, n_pairs = gridDim.x / 2;
  int32_t* status = G.status;
  constexpr uint32_t TMEM_COLS = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      tc::mbar_init(full(s), 1);                 // leader: its producer's arrival + both CTAs' transaction bytes
      tc::mbar_init(empty(s), 1);                // one commit arrival (sent to both CTAs)
    }
    for (int a = 0; a < 2; ++a) {
      tc::mbar_init(acc_full(a), 1);
      tc::mbar_init(acc_empty(a), 256);          // leader: the epilogue threads of both CTAs
    }
    tc::fence_barrier_init();
  }
  if (warp == 1) {
    tc::tmem_alloc2(slot, TMEM_COLS);
    tc::tmem_relinquish2();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();                        // the peer's barriers exist before anything signals them
  tc::tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(slot));
  pdl_launch_dependents();

  if (warp == 0 && lane == 0) {
    // ---- TMA producer (both CTAs): own A rows, own half of B's columns; bytes counted on the leader's barrier ----
    int it = 0;
    bool ok = true;
    TileCoord tcd;
    pdl_wait();
    for (int w = pair_id; ok && pair_tile_at(G, w, &tcd); w += n_pairs) {
      const TcProblem& P = G.p[tcd.prob];
      const int m0 = tcd.m0 + (int)rank * 128, n0 = tcd.n0 + (int)rank * 128;
      for (int t = 0; t < P.n_terms && ok; ++t) {
        const int kb_begin = t == 0 ? tcd.kb0 : 0, kb_end = t == 0 ? tcd.kb1 : P.kblocks[t];
        for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          const uint32_t sa = base + s * SP::STAGE, sb = sa + SP::A_BYTES;
          if (!tc::mbar_wait(empty(s), ph ^ 1, status, 111)) { ok = false; break; }
          if (rank == 0) tc::mbar_expect_tx(full(s), 2 * SP::STAGE);
          const uint32_t fb = tc::map_to_cta(full(s), 0);
          if (P.a_mn[t]) tc::tma_load_3d_pair(sa, &P.ta[t], fb, 0, kb * BK, m0 / 64);
          else tc::tma_load_3d_pair(sa, &P.ta[t], fb, 0, m0, kb);
          if (P.b_mn[t]) tc::tma_load_3d_pair(sb, &P.tb[t], fb, 0, kb * BK, n0 / 64);
          else tc::tma_load_3d_pair(sb, &P.tb[t], fb, 0, n0, kb);
        }
      }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ---- MMA issuer (leader only) --------------------------------------------------------------
    int s = 0, ti = 0;
    uint32_t ph = 0;
    bool ok = true;
    TileCoord tcd;
    const uint32_t hi = tc::smem_desc_hi(1024);
    for (int w = pair_id; ok && pair_tile_at(G, w, &tcd); w += n_pairs, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      if (!tc::mbar_wait(acc_empty(ab), ((ti >> 1) & 1) ^ 1, status, 114)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t d_tmem = tmem_base + ab * BN;
      uint32_t acc = 0;
      for (int t = 0; t < P.n_terms && ok; ++t) {
        const uint32_t idesc = tc::idesc_bf16(256, BN, P.a_mn[t], P.b_mn[t]);
        const uint32_t a_lo0 = tc::smem_desc_lo(base, P.a_mn[t] ? 8192u : 16u), a_step = P.a_mn[t] ? 128u : 2u;
        const uint32_t b_lo0 = tc::smem_desc_lo(base + SP::A_BYTES, P.b_mn[t] ? 8192u : 16u), b_step = P.b_mn[t] ? 128u : 2u;
        const int nkb = t == 0 ? tcd.kb1 - tcd.kb0 : P.kblocks[t];
        for (int kb = 0; kb < nkb; ++kb) {
          if (!tc::mbar_wait(full(s), ph, status, 112)) { ok = false; break; }
          tc::tc_fence_after();
          uint32_t a_lo = a_lo0 + (uint32_t)s * (SP::STAGE >> 4), b_lo = b_lo0 + (uint32_t)s * (SP::STAGE >> 4);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            tc::mma_bf16_ss_w2(d_tmem, a_lo, hi, b_lo, hi, idesc, acc);
            acc = 1;
            a_lo += a_step; b_lo += b_step;
          }
          tc::mma_commit2_both(empty(s));        // frees the stage in both CTAs once these MMAs have read it
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
      if (ok) tc::mma_commit2_both(acc_full(ab));
    }
  } else if (warp >= 2) {
    // ---- epilogue (both CTAs): this CTA's 128 accumulator rows, as in the single-CTA kernel -------------
    pdl_wait();
    group_chores(G, threadIdx.x - 64, 128);
    const int q = warp % 4;
    const int r = q * 32 + lane;
    int ti = 0, pc = 0;
    bool ok = true;
    TileCoord tcd;
    for (int w = pair_id; ok && pair_tile_at(G, w, &tcd); w += n_pairs, ++ti) {
      const TcProblem& P = G.p[tcd.prob];
      const int ab = ti & 1;
      const int m0 = tcd.m0 + (int)rank * 128;
      const int row = m0 + r;
      const bool pad = P.t_pad > 0 && (row % P.t_pad) >= P.seq;
      const bool has_res = P.residual && row < P.m;
      uint4 rv[8];
      if (has_res) {
        const __nv_bfloat16* rp = P.residual + ((long long)(tcd.n0 / 64) * P.c_rpad + row) * 64;
#pragma unroll
        for (int j = 0; j < 8; ++j) rv[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
      }
      const float* bias = P.bias;
      float bl[BN / 32];
      if (bias) {
#pragma unroll
        for (int k = 0; k < BN / 32; ++k) {
          const int c = tcd.n0 + lane * (BN / 32) + k;
          bl[k] = c < P.n ? bias[c] : 0.f;
        }
      }
      if (!tc::mbar_wait(acc_full(ab), (ti >> 1) & 1, status, 113)) { ok = false; break; }
      tc::tc_fence_after();
      float dot_acc = 0.f;
#pragma unroll 1
      for (int pn = 0; pn < BN / 64; ++pn) {
        const int n = tcd.n0 + pn * 64;
        if (n >= P.n) break;
        uint32_t v[64];
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64, *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
        tc::tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + pn * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
        tc::tmem_ld_wait();
        if (P.ksplit > 1) {
#pragma unroll 1
          for (int hf = 0; hf < 2; ++hf) {
            const uint32_t stg = base + SP::STG_OFF + (uint32_t)(q * 2 + (pc & 1)) * 4096u;
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)j ^ (uint32_t)(lane & 7)) * 16)),
                           "r"(hf ? v[32 + 4 * j] : v[4 * j]), "r"(hf ? v[33 + 4 * j] : v[4 * j + 1]),
                           "r"(hf ? v[34 + 4 * j] : v[4 * j + 2]), "r"(hf ? v[35 + 4 * j] : v[4 * j + 3]) : "memory");
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tc::tma_reduce_add_4d(&P.tacc, stg, 0, hf, m0 + q * 32, n / 64);
              tc::bulk_commit_group();
              tc::bulk_wait_group_read1();
            }
            ++pc;
          }
          continue;
        }
        uint4 outv[8];
        uint32_t* ow = reinterpret_cast<uint32_t*>(outv);
        if (has_res) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const __nv_bfloat16* rb = reinterpret_cast<const __nv_bfloat16*>(&rv[j]);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[8 * j + k] = __float_as_uint(__uint_as_float(v[8 * j + k]) + __bfloat162float(rb[k]));
          }
          if (pn + 1 < BN / 64 && n + 64 < P.n) {
            const __nv_bfloat16* rp = P.residual + ((long long)(n / 64 + 1) * P.c_rpad + row) * 64;
#pragma unroll
            for (int j = 0; j < 8; ++j) rv[j] = *reinterpret_cast<const uint4*>(rp + 8 * j);
          }
        }
        if (bias) {
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            const float b0 = __shfl_sync(0xffffffffu, bl[j % (BN / 32)], (pn * 64 + j) / (BN / 32));
            const float b1 = __shfl_sync(0xffffffffu, bl[(j + 1) % (BN / 32)], (pn * 64 + j + 1) / (BN / 32));
            ow[j / 2] = tc::pack_bf16(pad ? 0.f : __uint_as_float(v[j]) + b0, pad ? 0.f : __uint_as_float(v[j + 1]) + b1);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 64; j += 2)
            ow[j / 2] = tc::pack_bf16(pad ? 0.f : __uint_as_float(v[j]), pad ? 0.f : __uint_as_float(v[j + 1]));
        }
        if (P.dot_with && row < P.m) {
          const __nv_bfloat16* ap = P.dot_with + ((long long)(n / 64) * P.c_rpad + row) * 64;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 av = *reinterpret_cast<const uint4*>(ap + 8 * j);
            const __nv_bfloat16* ab16 = reinterpret_cast<const __nv_bfloat16*>(&av);
#pragma unroll
            for (int k = 0; k < 8; k += 2) {
              const uint32_t w2 = ow[4 * j + k / 2];
              dot_acc = fmaf(__uint_as_float(w2 << 16), __bfloat162float(ab16[k]), dot_acc);
              dot_acc = fmaf(__uint_as_float(w2 & 0xffff0000u), __bfloat162float(ab16[k + 1]), dot_acc);
            }
          }
          if ((n + 64) % P.dot_hd == 0) {
            const int hh = n / P.dot_hd, bb = row / P.t_pad, tt = row % P.t_pad;
            P.dot_out[((long long)bb * P.dot_hq + hh) * P.t_pad + tt] = dot_acc;
            dot_acc = 0.f;
          }
        }
        const uint32_t stg = base + SP::STG_OFF + (uint32_t)(q * 2 + (pc & 1)) * 4096u;
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + lane * 128 + (((uint32_t)j ^ (uint32_t)(lane & 7)) * 16)),
                       "r"(outv[j].x), "r"(outv[j].y), "r"(outv[j].z), "r"(outv[j].w) : "memory");
        tc::fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          tc::tma_store_3d(&P.tc, stg, 0, m0 + q * 32, n / 64);
          tc::bulk_commit_group();
          tc::bulk_wait_group_read1();
        }
        ++pc;
      }
      tc::tc_fence_before();
      tc::mbar_arrive_cluster(tc::map_to_cta(acc_empty(ab), 0));     // the leader's barrier, from either CTA
    }
    if (lane == 0) tc::bulk_wait_group0();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync_all();                        // neither CTA frees tensor memory or leaves while its peer may still
  if (warp == 1) tc::tmem_dealloc2(tmem_base, TMEM_COLS);   // read its shared memory or signal its barriers
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

// Self-test of the bounded wait every tensor-core kernel relies on: one block initialises an mbarrier that nothing
// ever signals and waits on it through the same tc::mbar_wait, with a short limit.  The wait must give up, record
// its code in the status word and let the block return normally.
__global__ void wait_timeout_selftest_kernel(int32_t* status, long long limit_cycles) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);
    tc::fence_barrier_init();
  }
  __syncthreads();
  const bool ok = tc::mbar_wait(tc::smem_u32(&bar), 0, status, 901, limit_cycles);
  __syncthreads();
  if (threadIdx.x == 0) status[1] = ok ? 2 : 1;     // the block reached its normal end
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(int32_t* status, long long limit_cycles, cudaStream_t st) {
  wait_timeout_selftest_kernel<<<1, 64, 0, st>>>(status, limit_cycles);
  return cudaGetLastError();
}

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
bool fbl_encode_f32_panel_map(CUtensorMap* map, const void* base, int64_t r_pad, int panels, int box_rows, int box_halves) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {32, 2, (cuuint64_t)r_pad, (cuuint64_t)panels};
  cuuint64_t strides[3] = {128, 256, (cuuint64_t)r_pad * 256};
  cuuint32_t box[4] = {32, (cuuint32_t)box_halves, (cuuint32_t)box_rows, 1};
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

// Problem set-up shared by the two kernels: tensor maps, operand orientations, epilogue extras and reduction
// slices of every problem of a launch.  bn_box: columns of B one CTA loads per k-block; tile_m x tile_n: the output
// tile a work unit covers (the CTA pair's 256 x 256, or one CTA's 128 x BN).  Returns the number of work units in
// *units.
cudaError_t fill_group(TcGroup& G, const GemmArgs* gs, int count, int32_t* status, int bn_box, int tile_m, int tile_n,
                       int* units) {
  memset(&G, 0, sizeof(G));
  G.count = count;
  G.status = status;
  G.zero_ptr = (uint4*)gs[0].zero_ptr; G.zero_vec = (long long)(gs[0].zero_bytes / 16); G.reset_status = gs[0].reset_status;
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
      if (tm.b_trans) ok = fbl_encode_rtile_map(&P.tb[t], tm.b, tm.b_rpad, tm.k / 64, bn_box, 1);
      else ok = fbl_encode_rtile_map(&P.tb[t], tm.b, tm.b_rpad, g.n / 64, BK, bn_box / 64);
      if (!ok) return cudaErrorInvalidValue;
    }
    P.m = g.m; P.n = g.n;
    if (!fbl_encode_rtile_map(&P.tc, g.c, g.c_rpad, g.n / 64, 32, 1)) return cudaErrorInvalidValue;   // one warp's rows
    P.b_static = g.b_static;
    P.c = (__nv_bfloat16*)g.c; P.c_rpad = g.c_rpad;
    P.bias = g.bias; P.residual = (const __nv_bfloat16*)g.residual;
    P.seq = g.seq; P.t_pad = g.t_pad;
    P.dot_with = (const __nv_bfloat16*)g.dot_with; P.dot_out = g.dot_out; P.dot_hd = g.dot_hd; P.dot_hq = g.dot_hq;
    P.epi = g.epi; P.aux1 = (const __nv_bfloat16*)g.aux1;
    if (g.epi != 0) {
      if (g.epi < 1 || g.epi > 4 || g.ksplit > 1 || g.dot_with || (g.epi >= 2 && !g.residual) || (g.epi == 4 && !g.aux1) ||
          (g.epi != 2 && !g.c2))
        return cudaErrorInvalidValue;
      if (g.epi != 2 && !fbl_encode_rtile_map(&P.tc2, g.c2, g.c_rpad, g.n / 64, 32, 1)) return cudaErrorInvalidValue;
    }
    P.ksplit = 1;
    if (g.ksplit > 1) {
      if (g.n_terms != 1 || g.bias || g.residual || g.dot_with || g.t_pad > 0 || !g.acc) return cudaErrorInvalidValue;
      const int per = (P.kblocks[0] + g.ksplit - 1) / g.ksplit;        // no empty slice
      P.ksplit = (P.kblocks[0] + per - 1) / per;
      if (!fbl_encode_f32_panel_map(&P.tacc, g.acc, g.c_rpad, g.n / 64, 32, 1)) return cudaErrorInvalidValue;
    }
    tiles += ((g.m + tile_m - 1) / tile_m) * ((g.n + tile_n - 1) / tile_n) * P.ksplit;
  }
  *units = tiles;
  return cudaSuccess;
}

template <int BN, int STAGES>
cudaError_t launch_group_bn(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st, int esets_choice) {
  TcGroup G;
  int tiles = 0;
  cudaError_t e = fill_group(G, gs, count, status, BN, BM, BN, &tiles);
  if (e != cudaSuccess) return e;
  using SP = SmemPlan<BN, STAGES>;
  const int grid = tiles < p->sm_count ? tiles : p->sm_count;
  // one tile per block at most: the epilogue is exposed, and the variant with two sets of epilogue warps halves it
  // (with several tiles per block the epilogues overlap the next main loops and the extra warps only cost)
  const int esets_knob = esets_choice ? esets_choice : p->knob_gemm_esets;
  const bool two_sets = esets_knob ? esets_knob == 2 : tiles <= p->sm_count;
  bool epi = false;
  for (int i = 0; i < count; ++i) epi = epi || gs[i].epi != 0;
  if (epi) {                       // the variant with the fused activations (feed-forward block only)
    if (two_sets) {
      auto k = gemm_tc_kernel<BN, STAGES, 2, true>;
      cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
      if (attr_err != cudaSuccess) return attr_err;
      return launch_pdl(k, dim3(grid), dim3(320), SP::TOTAL, st, G);
    }
    auto k = gemm_tc_kernel<BN, STAGES, 1, true>;
    cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
    if (attr_err != cudaSuccess) return attr_err;
    return launch_pdl(k, dim3(grid), dim3(192), SP::TOTAL, st, G);
  }
  if (two_sets) {
    auto k = gemm_tc_kernel<BN, STAGES, 2>;
    cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
    if (attr_err != cudaSuccess) return attr_err;
    return gs[0].serial ? launch_serial(k, dim3(grid), dim3(320), SP::TOTAL, st, G)
                        : launch_pdl(k, dim3(grid), dim3(320), SP::TOTAL, st, G);
  }
  auto k = gemm_tc_kernel<BN, STAGES, 1>;
  cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
  if (attr_err != cudaSuccess) return attr_err;
  return gs[0].serial ? launch_serial(k, dim3(grid), dim3(192), SP::TOTAL, st, G)
                      : launch_pdl(k, dim3(grid), dim3(192), SP::TOTAL, st, G);
}

cudaError_t launch_group_pair(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st) {
  TcGroup G;
  int tiles = 0;
  cudaError_t e = fill_group(G, gs, count, status, 128, 256, 256, &tiles);   // each CTA loads 128 of the pair's 256 columns
  if (e != cudaSuccess) return e;
  using SP = PairSmem;
  auto k = gemm_tc_pair_kernel;
  cudaError_t attr_err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SP::TOTAL);
  if (attr_err != cudaSuccess) return attr_err;
  const int pairs = tiles < p->sm_count / 2 ? tiles : p->sm_count / 2;
  return gs[0].serial ? launch_serial(k, dim3(2 * pairs), dim3(192), SP::TOTAL, st, G)
                      : launch_pdl(k, dim3(2 * pairs), dim3(192), SP::TOTAL, st, G);
}

cudaError_t launch_gemm_tc_group(const fbl_plan* p, const GemmArgs* gs, int count, int32_t* status, cudaStream_t st,
                                 int launch_id) {
  if (count < 1 || count > MAX_PROBLEMS) return cudaErrorInvalidValue;
  fbl_plan::GemmChoice ch = {0, -1, 0};
  if (launch_id >= 0 && launch_id < FBL_GEMM_LAUNCH_COUNT) ch = p->choice[launch_id];
  bool wide = true;                       // 128 x 256 tiles when every problem's N is whole 256-column blocks
  int tiles_wide = 0;
  for (int i = 0; i < count; ++i) {
    wide = wide && gs[i].n % 256 == 0;
    for (int t = 0; t < gs[i].n_terms; ++t)
      if (gs[i].t[t].b_trans && gs[i].t[t].b_rpad < 256) wide = false;
    tiles_wide += ((gs[i].m + BM - 1) / BM) * ((gs[i].n + 255) / 256) * (gs[i].ksplit > 1 ? gs[i].ksplit : 1);
  }
  const bool wide_legal = wide;
  // with too few wide tiles to occupy the SMs, narrower tiles (twice as many) finish sooner
  if (wide && tiles_wide * 3 < p->sm_count * 2) wide = false;
  // CTA pairs on 256 x 256 tiles for large problems (several rounds of tiles per SM pair): measured 2-6 % faster
  // on the workload 5 GEMMs, no gain or a loss below that
  bool any_epi = false;
  for (int i = 0; i < count; ++i) any_epi = any_epi || gs[i].epi != 0;
  // an offline choice for this launch overrides the heuristics below wherever its tile shape is legal
  if (ch.bn == 128) wide = false;
  else if (ch.bn == 256 && wide_legal) wide = true;
  const int pair_mode = ch.pair >= 0 ? ch.pair : p->knob_gemm_pair;       // 0 never, 1 whenever legal, -1 by size
  if (pair_mode == 1 && wide_legal && !any_epi) return launch_group_pair(p, gs, count, status, st);
  if (wide && pair_mode != 0 && !any_epi) {
    long long pair_tiles = 0;
    for (int i = 0; i < count; ++i)
      pair_tiles += (long long)((gs[i].m + 255) / 256) * (gs[i].n / 256) * (gs[i].ksplit > 1 ? gs[i].ksplit : 1);
    if (pair_tiles >= 4 * (p->sm_count / 2)) return launch_group_pair(p, gs, count, status, st);
  }
  if (wide) return launch_group_bn<256, 4>(p, gs, count, status, st, ch.esets);
  return launch_group_bn<128, 6>(p, gs, count, status, st, ch.esets);
}

// How many slices to cut the reduction loops of the splittable problems of a group into (the same number for all
// of them).  The persistent kernel deals work units to its blocks round-robin, so a few long units beside many
// short ones leave most SMs idle: this replays the dealing for each candidate and keeps the one whose longest
// block finishes first, charging the fp32 detour (zero-fill, bulk reductions, rounding pass) as extra k-blocks.
int gemm_tc_choose_split(int sm_count, const GemmShape* sh, int count) {
  static const int cand[] = {1, 2, 3, 4, 6, 8, 12, 16};
  double base_cost = 0.0, best_cost = 0.0;
  int best = 1;
  for (int ci = 0; ci < (int)(sizeof(cand) / sizeof(cand[0])); ++ci) {
    const int S = cand[ci];
    bool wide = true;
    long long tiles_wide = 0;
    bool any_split = false;
    for (int i = 0; i < count; ++i) {
      wide = wide && sh[i].n % 256 == 0;
      const int s_i = (sh[i].splittable && S > 1) ? S : 1;
      if (s_i > 1 && sh[i].kblocks / s_i < 8) { any_split = false; tiles_wide = -1; break; }   // slices too short
      any_split = any_split || s_i > 1;
      tiles_wide += (long long)((sh[i].m + BM - 1) / BM) * ((sh[i].n + 255) / 256) * s_i;
    }
    if (tiles_wide < 0 || (S > 1 && !any_split)) continue;
    if (wide && tiles_wide * 3 < (long long)sm_count * 2) wide = false;
    const int bn = wide ? 256 : 128;
    const double per_kb = wide ? 1.32 : 1.0;               // a k-block of a 128 x 256 tile takes about 660 clk, of 128 x 128 about 500
    long long units = 0;
    for (int i = 0; i < count; ++i)
      units += (long long)((sh[i].m + BM - 1) / BM) * ((sh[i].n + bn - 1) / bn) * ((sh[i].splittable && S > 1) ? S : 1);
    const int grid = (int)(units < sm_count ? units : sm_count);
    std::vector<double> load((size_t)grid, 0.0);
    long long w = 0;
    for (int i = 0; i < count; ++i) {
      const int s_i = (sh[i].splittable && S > 1) ? S : 1;
      const long long n_i = (long long)((sh[i].m + BM - 1) / BM) * ((sh[i].n + bn - 1) / bn) * s_i;
      const double len = ((sh[i].kblocks + s_i - 1) / s_i + (s_i > 1 ? 2 : 0) + 3) * per_kb;   // + pipeline fill and epilogue
      for (long long u = 0; u < n_i; ++u, ++w) load[w % grid] += len;
    }
    double mk = 0;
    for (int b = 0; b < grid; ++b) mk = load[b] > mk ? load[b] : mk;
    if (S > 1) mk += 16;                                   // zero-fill and rounding pass
    if (ci == 0) { base_cost = mk; best_cost = mk; }
    else if (mk < 0.85 * base_cost && mk < best_cost) { best = S; best_cost = mk; }   // worth it only with a clear gain
  }
  return best;
}
