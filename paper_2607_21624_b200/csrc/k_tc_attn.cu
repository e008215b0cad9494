// Fused attention on tcgen05 tensor cores, operands in R-Tile order fetched by TMA.
//
// Forward: one block per (128-query tile, head, batch).  S = Q K^T goes to TMEM (two buffers, so the
// tensor pipe computes the next score tile while the softmax warps work on the current one); the
// softmax warps own one query row per thread, keep the running max / sum, and hand P (bf16) to the
// tensor pipe in tensor memory, over the score columns it was computed from; O accumulates in TMEM and is
// rescaled in place only when a row's running max moved.  K/V tiles of the group's KV head are addressed by the head map
// g = h / G; the head split of Q, K, V and the merge of O are column-panel coordinates of the TMA
// boxes and of the output rows, no data is rearranged.
#include <string.h>

#include <type_traits>

#include "attn_common.cuh"
#include "fbl_internal.h"
#include "pdl.cuh"
#include "tc_common.cuh"

namespace {

constexpr int BQ = 128, BKV = 128;
constexpr float LOG2E = 1.4426950408889634f;

struct alignas(64) AttnFwdParams {
  CUtensorMap tq, tk, tv;
  __nv_bfloat16* a;      // merged-head output [n_pad, dq] in R-Tile order
  float* lse;            // [B, Hq, t_pad]
  long long n_pad;
  int seq, t_pad, hq, group, causal;
  int seq_k, t_pad_k;    // key-side sequence length and padded length (those of the query side in self-attention)
  int pair;              // 1: each block owns two adjacent query tiles, one per softmax warp group
  int batch, n_slots, chunk;   // grid = n_slots * hq * batch blocks, see decode_block
  float scale;
  int32_t* status;
};

template <int HD, int TILES>
struct FwdSmem {
  static constexpr uint32_t PANELS = HD / 64;
  static constexpr uint32_t TILE = PANELS * 16384;          // 128 rows x HD bf16
  static constexpr uint32_t Q_OFF = 0;                      // TILES query tiles
  static constexpr uint32_t K_OFF = TILES * TILE;           // 2 stages
  static constexpr uint32_t V_OFF = (TILES + 2) * TILE;     // 2 stages
  static constexpr uint32_t BAR_OFF = (TILES + 4) * TILE;
  static constexpr uint32_t N_BARS = 18;
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16;
};

enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_PFULL = 12, B_PVDONE = 15 };   // SFULL, PFULL: one per score buffer (up to 3)

// warp 0 TMA, warp 1 MMA, then one softmax warp group (4 warps) per query tile of the block.  TILES = 2: two
// adjacent query tiles share the K/V tiles, one block per SM.  TILES = 1 (head_dim 64 only: its tiles leave room): a
// block of 192 threads with one query tile, half the tensor memory and at most 128 registers per thread, so that two
// blocks share an SM and one's set-up and epilogue overlap the other's key loop (short sequences are mostly that).

// A row's running max is only raised (and O rescaled) when the new max exceeds it by more than this many
// powers of two; until then the probabilities are computed against the stale max and stay below 2^8.
constexpr float RESCALE_LOG2 = 8.f;

template <int HD, int TILES>
__global__ void __launch_bounds__(64 + 128 * TILES, TILES == 1 ? 2 : 1) attn_fwd_tc_kernel(const __grid_constant__ AttnFwdParams P) {
  using SM = FwdSmem<HD, TILES>;
  constexpr uint32_t PANELS = SM::PANELS;
  // Score buffers in tensor memory.  HD = 128 (and one-tile blocks): one per query tile, P written over S, so the
  // next S of a tile follows its P V product.  HD = 64 with two tiles leaves room for a third buffer (3 x 128 score
  // columns + 2 x 64 output columns = 512): the block's work items (tile, key tile), in issue order, then take the
  // buffers in rotation, item n using buffer n % 3, and the S product of item n + 3 is issued right after the P V
  // product of item n.  Every warp group then finds its next scores computed when it finishes a tile, instead of
  // waiting for P V and S behind its own P.
  constexpr bool ROT = TILES == 2 && HD == 64;
  constexpr int NBUF = ROT ? 3 : TILES;
  constexpr uint32_t O_COL = 128 * NBUF, TMEM_COLS = 256 * TILES;   // score buffer i at 128 i, O of tile g at O_COL + HD g
  static_assert(O_COL + TILES * HD <= TMEM_COLS, "tensor memory columns");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = tc::smem_u32(smem_raw);
  const uint32_t bars = base + SM::BAR_OFF;
  const uint32_t slot = bars + 8 * SM::N_BARS;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int n_qt = (P.seq + BQ - 1) / BQ;
  int slot_i, hb;
  decode_block((int)blockIdx.x, P.n_slots, P.hq * P.batch, P.chunk, &slot_i, &hb);
  const int h = hb % P.hq, b = hb / P.hq, g = h / P.group;
  const int row0 = b * P.t_pad, row0k = b * P.t_pad_k;     // first row of this sequence on the query and key sides
  int32_t* status = P.status;
  // with pairing a block owns two adjacent tiles, whose key ranges differ by one tile, so both warp groups stay
  // busy for the whole loop
  const int slot_x = P.n_slots - 1 - slot_i;                 // heaviest (latest) causal tiles first
  const bool pair = TILES == 2 && P.pair;
  const int qt0 = pair ? min(2 * slot_x + 1, n_qt - 1) : slot_x;
  const int qt1 = (pair && 2 * slot_x + 1 < n_qt) ? 2 * slot_x : -1;   // odd tile count: the last block has one tile
  auto kv_tiles = [&](int t) {
    const int kv_end = t < 0 ? 0 : (P.causal ? min(P.seq_k, (t + 1) * BQ) : P.seq_k);
    return (kv_end + BKV - 1) / BKV;
  };
  const int n_kv0 = kv_tiles(qt0), n_kv1 = kv_tiles(qt1);
  const int n_kv_max = max(n_kv0, n_kv1);
  if ((base & 1023u) != 0) {
    if (threadIdx.x == 0) atomicCAS(status, 0, 299);
    return;
  }

  if (threadIdx.x == 0) {
    tc::mbar_init(bar(B_QFULL), 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(bar(B_KFULL + s), 1);
      tc::mbar_init(bar(B_KEMPTY + s), 1);
      tc::mbar_init(bar(B_VFULL + s), 1);
      tc::mbar_init(bar(B_VEMPTY + s), 1);
      tc::mbar_init(bar(B_PVDONE + s), 1);
    }
    for (int s = 0; s < 3; ++s) {
      tc::mbar_init(bar(B_SFULL + s), 1);
      tc::mbar_init(bar(B_PFULL + s), 128);
    }
    tc::fence_barrier_init();
    // This thread is the TMA producer: once the kernel before this one (which writes Q, K, V) is complete, the
    // query tiles and the first K / V tiles are requested right here, so that their latency overlaps the
    // tensor-memory allocation and the block-wide barrier below.
    tc::tma_prefetch_desc(&P.tq);
    tc::tma_prefetch_desc(&P.tk);
    tc::tma_prefetch_desc(&P.tv);
    pdl_wait();
    tc::mbar_expect_tx(bar(B_QFULL), (qt1 >= 0 ? 2u : 1u) * SM::TILE);
    tc::tma_load_3d(base + SM::Q_OFF, &P.tq, bar(B_QFULL), 0, row0 + qt0 * BQ, h * (int)PANELS);
    if (qt1 >= 0) tc::tma_load_3d(base + SM::Q_OFF + SM::TILE, &P.tq, bar(B_QFULL), 0, row0 + qt1 * BQ, h * (int)PANELS);
    if (n_kv_max > 0) {
      tc::mbar_expect_tx(bar(B_KFULL), SM::TILE);
      tc::tma_load_3d(base + SM::K_OFF, &P.tk, bar(B_KFULL), 0, row0k, g * (int)PANELS);
      tc::mbar_expect_tx(bar(B_VFULL), SM::TILE);
      tc::tma_load_3d(base + SM::V_OFF, &P.tv, bar(B_VFULL), 0, row0k, g * (int)PANELS);
    }
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
    // ---- TMA producer (the query tiles and key tile 0 were requested during set-up) ---------------
    for (int j = 1; j < n_kv_max; ++j) {
      const int s = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      if (!tc::mbar_wait(bar(B_KEMPTY + s), ph ^ 1, status, 201)) break;
      tc::mbar_expect_tx(bar(B_KFULL + s), SM::TILE);
      tc::tma_load_3d(base + SM::K_OFF + s * SM::TILE, &P.tk, bar(B_KFULL + s), 0, row0k + j * BKV, g * (int)PANELS);
      if (!tc::mbar_wait(bar(B_VEMPTY + s), ph ^ 1, status, 202)) break;
      tc::mbar_expect_tx(bar(B_VFULL + s), SM::TILE);
      tc::tma_load_3d(base + SM::V_OFF + s * SM::TILE, &P.tv, bar(B_VFULL + s), 0, row0k + j * BKV, g * (int)PANELS);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer --------------------------------------------------------------------------
    // Per key tile j: [P0(j) ready] PV0(j), S0(j+1), [P1(j) ready] PV1(j), S1(j+1): while one warp group works
    // on its scores the tensor pipe serves the other one.  S and P of a query tile share TMEM columns, so
    // S(j+1) is issued after PV(j), which reads P(j) (the tensor pipe executes in issue order).
    const uint32_t idesc_s = tc::idesc_bf16(BQ, BKV, 0, 0);          // Q K-major, K K-major
    const uint32_t idesc_o = tc::idesc_bf16(BQ, HD, 0, 1);           // P from TMEM, V MN-major (rows are keys)
    // Descriptor words are formed once; per instruction only the start-address field of the low word moves.
    const uint32_t hi = tc::smem_desc_hi(1024);
    const uint32_t q_lo = tc::smem_desc_lo(base + SM::Q_OFF, 16), k_lo = tc::smem_desc_lo(base + SM::K_OFF, 16);
    const uint32_t v_lo = tc::smem_desc_lo(base + SM::V_OFF, 16384);
    auto issue_s = [&](int w, int j) {
      const uint32_t ql = q_lo + w * (SM::TILE >> 4), kl = k_lo + (j & 1) * (SM::TILE >> 4);
#pragma unroll
      for (uint32_t kk = 0; kk < HD / 16; ++kk) {
        const uint32_t o = (kk / 4) * 1024 + (kk % 4) * 2;            // 16-byte units: 64-column panel, 16-element step
        tc::mma_bf16_ss_w(tmem_base + w * 128, ql + o, hi, kl + o, hi, idesc_s, kk > 0);
      }
      tc::mma_commit(bar(B_SFULL + w));
    };
    auto issue_pv = [&](int w, int j) {
      const uint32_t vl = v_lo + (j & 1) * (SM::TILE >> 4);
#pragma unroll
      for (uint32_t kk = 0; kk < BKV / 16; ++kk) {
        // A operand from tensor memory: the packed bf16 P row of each lane, 16 keys = 8 columns per step
        tc::mma_bf16_ts_w(tmem_base + O_COL + w * HD, tmem_base + w * 128 + kk * 8, vl + kk * 128, hi, idesc_o,
                          (j > 0 || kk > 0) ? 1u : 0u);
      }
      tc::mma_commit(bar(B_PVDONE + w));
    };
    if constexpr (ROT) {
      // Work items in issue order: (tile 0, j), (tile 1, j) while tile 1 has key tiles, then tile 0's remaining
      // ones (n_kv0 >= n_kv1: tile 0 is the later query tile).  Barriers of a score buffer are used once per
      // rotation, so neither side can run more than one phase ahead on any of them.
      const int n_items = n_kv0 + n_kv1;
      auto item = [&](int n, int& w, int& j) {
        if (n < 2 * n_kv1) { w = n & 1; j = n >> 1; } else { w = 0; j = n - n_kv1; }
      };
      auto issue_s_item = [&](int n) -> bool {
        int w, j; item(n, w, j);
        // tile 0 is the first user of every key tile, and the last one where tile 1 has none
        if (w == 0 && !tc::mbar_wait(bar(B_KFULL + (j & 1)), (j >> 1) & 1, status, 205)) return false;
        const uint32_t ql = q_lo + w * (SM::TILE >> 4), kl = k_lo + (j & 1) * (SM::TILE >> 4);
        const uint32_t d = tmem_base + (uint32_t)(n % 3) * 128;
#pragma unroll
        for (uint32_t kk = 0; kk < HD / 16; ++kk) {
          const uint32_t o = (kk / 4) * 1024 + (kk % 4) * 2;
          tc::mma_bf16_ss_w(d, ql + o, hi, kl + o, hi, idesc_s, kk > 0);
        }
        tc::mma_commit(bar(B_SFULL + n % 3));
        if (w == 1 || j >= n_kv1) tc::mma_commit(bar(B_KEMPTY + (j & 1)));
        return true;
      };
      bool ok = tc::mbar_wait(bar(B_QFULL), 0, status, 203);
      if (ok) tc::tc_fence_after();
      for (int n = 0; n < 3 && n < n_items && ok; ++n) ok = issue_s_item(n);
      for (int n = 0; n < n_items && ok; ++n) {
        int w, j; item(n, w, j);
        if (w == 0 && !tc::mbar_wait(bar(B_VFULL + (j & 1)), (j >> 1) & 1, status, 207)) { ok = false; break; }
        if (!tc::mbar_wait(bar(B_PFULL + n % 3), (n / 3) & 1, status, 206)) { ok = false; break; }
        tc::tc_fence_after();
        const uint32_t vl = v_lo + (j & 1) * (SM::TILE >> 4);
        const uint32_t pa = tmem_base + (uint32_t)(n % 3) * 128, od = tmem_base + O_COL + w * HD;
#pragma unroll
        for (uint32_t kk = 0; kk < BKV / 16; ++kk)
          tc::mma_bf16_ts_w(od, pa + kk * 8, vl + kk * 128, hi, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
        tc::mma_commit(bar(B_PVDONE + w));
        if (w == 1 || j >= n_kv1) tc::mma_commit(bar(B_VEMPTY + (j & 1)));
        if (n + 3 < n_items) ok = issue_s_item(n + 3);     // into the buffer whose P the product above has just read
      }
    } else {
    bool ok = tc::mbar_wait(bar(B_QFULL), 0, status, 203) && tc::mbar_wait(bar(B_KFULL), 0, status, 204);
    if (ok) {
      tc::tc_fence_after();
      if (n_kv0 > 0) issue_s(0, 0);
      if (TILES == 2 && n_kv1 > 0) issue_s(1, 0);
    }
    for (int j = 0; j < n_kv_max && ok; ++j) {
      const bool next = j + 1 < n_kv_max;
      if (!tc::mbar_wait(bar(B_VFULL + (j & 1)), (j >> 1) & 1, status, 207)) { ok = false; break; }
      if (next && !tc::mbar_wait(bar(B_KFULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, status, 205)) { ok = false; break; }
#pragma unroll
      for (int w = 0; w < TILES; ++w) {
        const int nk = w ? n_kv1 : n_kv0;
        if (ok && j < nk) {
          if (!tc::mbar_wait(bar(B_PFULL + w), j & 1, status, 206)) { ok = false; }
          else { tc::tc_fence_after(); issue_pv(w, j); }
        }
        if (ok && j + 1 < nk) issue_s(w, j + 1);
      }
      if (!ok) break;
      tc::mma_commit(bar(B_VEMPTY + (j & 1)));              // both P V products of this stage are behind us
      if (next) tc::mma_commit(bar(B_KEMPTY + ((j + 1) & 1)));   // ... and both score products of the next stage
      if (j == 0) tc::mma_commit(bar(B_KEMPTY));            // stage 0 scores were issued before the loop
    }
    }
  } else if (warp >= 2) {
    // ---- softmax warp groups: group w owns query tile qt[w], one query row per thread --------------
    const int w = (warp - 2) / 4;
    const int q = warp % 4;
    const int r = q * 32 + lane;
    const int n_kvw = w ? n_kv1 : n_kv0;
    const int i0 = (w ? qt1 : qt0) * BQ;
    const int gi = i0 + r;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const uint32_t o_addr = lane_addr + O_COL + w * HD;
    const float c = P.scale * LOG2E;
    const float tau = RESCALE_LOG2 / c;              // the same threshold in raw score units
    pdl_wait();                                      // before this role writes anything
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kvw && ok; ++j) {
      const int j0 = j * BKV;
      // score buffer and barrier phase of this (tile, key tile): see the MMA issuer
      const int n_item = ROT ? (w ? 2 * j + 1 : j + min(j, n_kv1)) : j;
      const int sbuf = ROT ? n_item % 3 : w;
      const uint32_t sph = ROT ? (uint32_t)(n_item / 3) & 1u : (uint32_t)j & 1u;
      const uint32_t s_addr = lane_addr + (uint32_t)sbuf * 128;
      if (!tc::mbar_wait(bar(B_SFULL + sbuf), sph, status, 208)) { ok = false; break; }
      tc::tc_fence_after();
      const bool need_mask = (j0 + BKV > P.seq_k) || (P.causal && j0 + BKV - 1 > i0);
      float mx, alpha, mc;
      float2 sum01 = make_float2(0.f, 0.f), sum23 = sum01;
      const float2 c2 = make_float2(c, c);
      bool moved;
      if constexpr (TILES == 2) {
        // The row's 128 scores come into registers with one wait (one block per SM: a thread may hold them all):
        // the maximum, the exponentials and the packing then run without touching tensor memory again until
        // the packed P row is stored over the score columns.
        uint32_t sr[128];
  #pragma unroll
        for (int cc = 0; cc < 4; ++cc) tc::tmem_ld32(s_addr + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[cc * 32]));
        tc::tmem_ld_wait();
        float* sv = reinterpret_cast<float*>(sr);
        if (need_mask) {
  #pragma unroll
          for (int k = 0; k < 128; ++k) {
            const int gj = j0 + k;
            if (gj >= P.seq_k || (P.causal && gj > gi)) sv[k] = -INFINITY;
          }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
  #pragma unroll
        for (int k = 0; k < 128; k += 8) {               // three-input maxima: one instruction per two scores
          mx0 = tc::fmax3(mx0, sv[k], sv[k + 1]); mx1 = tc::fmax3(mx1, sv[k + 2], sv[k + 3]);
          mx2 = tc::fmax3(mx2, sv[k + 4], sv[k + 5]); mx3 = tc::fmax3(mx3, sv[k + 6], sv[k + 7]);
        }
        mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        // lazy running max: move it only when the tile's max beats it by more than the threshold
        moved = mx > m + tau || m == -INFINITY;
        const float m_new = moved ? fmaxf(m, mx) : m;
        alpha = (m == -INFINITY) ? 0.f : tc::fast_exp2((m - m_new) * c);
        mc = (m_new == -INFINITY) ? 0.f : m_new * c;
        m = m_new;
        if (j > 0 && __any_sync(0xffffffffu, moved)) {
          // O is rescaled in place: the previous P V product must have finished
          if (!tc::mbar_wait(bar(B_PVDONE + w), (j - 1) & 1, status, 209)) { ok = false; break; }
          tc::tc_fence_after();
          const float a = moved ? alpha : 1.f;
  #pragma unroll 1
          for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t o[32];
            tc::tmem_ld32(o_addr + cc * 32, o);
            tc::tmem_ld_wait();
  #pragma unroll
            for (int k = 0; k < 32; k += 2) {
              const float2 v = __fmul2_rn(make_float2(__uint_as_float(o[k]), __uint_as_float(o[k + 1])), make_float2(a, a));
              o[k] = __float_as_uint(v.x); o[k + 1] = __float_as_uint(v.y);
            }
            tc::tmem_st32(o_addr + cc * 32, o);
          }
        }
        // P = exp2(S c - m c), its row sum, and P packed to bf16 (128 scores become 64 packed columns)
        const float2 nmc2 = make_float2(-mc, -mc);
  #pragma unroll
        for (int k = 0; k < 128; k += 4) {
          const float2 x01 = __ffma2_rn(make_float2(sv[k], sv[k + 1]), c2, nmc2);       // two-wide fp32 operations
          const float2 x23 = __ffma2_rn(make_float2(sv[k + 2], sv[k + 3]), c2, nmc2);
          const float p0 = tc::fast_exp2(x01.x), p1 = tc::fast_exp2(x01.y), p2 = tc::fast_exp2(x23.x), p3 = tc::fast_exp2(x23.y);
          sum01 = __fadd2_rn(sum01, make_float2(p0, p1)); sum23 = __fadd2_rn(sum23, make_float2(p2, p3));
          sr[k / 2] = tc::pack_bf16(p0, p1);
          sr[k / 2 + 1] = tc::pack_bf16(p2, p3);
        }
        tc::tmem_st32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
        tc::tmem_st32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
      } else {
        // At most 128 registers here (two blocks per SM): two passes over the scores in tensor memory, four
        // 32-column loads each, instead of holding the row.
        auto mask_chunk = [&](float* sc, int cc) {
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const int gj = j0 + cc * 32 + k;
            if (gj >= P.seq_k || (P.causal && gj > gi)) sc[k] = -INFINITY;
          }
        };
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t sr[32];
          tc::tmem_ld32(s_addr + cc * 32, sr);
          tc::tmem_ld_wait();
          float* sc = reinterpret_cast<float*>(sr);
          if (need_mask) mask_chunk(sc, cc);
#pragma unroll
          for (int k = 0; k < 32; k += 8) {
            mx0 = tc::fmax3(mx0, sc[k], sc[k + 1]); mx1 = tc::fmax3(mx1, sc[k + 2], sc[k + 3]);
            mx2 = tc::fmax3(mx2, sc[k + 4], sc[k + 5]); mx3 = tc::fmax3(mx3, sc[k + 6], sc[k + 7]);
          }
        }
        mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        moved = mx > m + tau || m == -INFINITY;
        const float m_new = moved ? fmaxf(m, mx) : m;
        alpha = (m == -INFINITY) ? 0.f : tc::fast_exp2((m - m_new) * c);
        mc = (m_new == -INFINITY) ? 0.f : m_new * c;
        m = m_new;
        if (j > 0 && __any_sync(0xffffffffu, moved)) {
          if (!tc::mbar_wait(bar(B_PVDONE + w), (j - 1) & 1, status, 209)) { ok = false; break; }
          tc::tc_fence_after();
          const float a = moved ? alpha : 1.f;
#pragma unroll 1
          for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t o[32];
            tc::tmem_ld32(o_addr + cc * 32, o);
            tc::tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; k += 2) {
              const float2 v = __fmul2_rn(make_float2(__uint_as_float(o[k]), __uint_as_float(o[k + 1])), make_float2(a, a));
              o[k] = __float_as_uint(v.x); o[k + 1] = __float_as_uint(v.y);
            }
            tc::tmem_st32(o_addr + cc * 32, o);
          }
        }
        const float2 nmc2 = make_float2(-mc, -mc);
        // pass 2: P packed to bf16 over the score columns already consumed (32 scores become 16 packed columns;
        // the thread owns the lane, so nobody else's data is overwritten)
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
          uint32_t sr[32];
          tc::tmem_ld32(s_addr + cc * 32, sr);
          tc::tmem_ld_wait();
          float* sc = reinterpret_cast<float*>(sr);
          if (need_mask) mask_chunk(sc, cc);
          uint32_t pk[16];
#pragma unroll
          for (int k = 0; k < 32; k += 4) {
            const float2 x01 = __ffma2_rn(make_float2(sc[k], sc[k + 1]), c2, nmc2);
            const float2 x23 = __ffma2_rn(make_float2(sc[k + 2], sc[k + 3]), c2, nmc2);
            const float p0 = tc::fast_exp2(x01.x), p1 = tc::fast_exp2(x01.y), p2 = tc::fast_exp2(x23.x), p3 = tc::fast_exp2(x23.y);
            sum01 = __fadd2_rn(sum01, make_float2(p0, p1)); sum23 = __fadd2_rn(sum23, make_float2(p2, p3));
            pk[k / 2] = tc::pack_bf16(p0, p1);
            pk[k / 2 + 1] = tc::pack_bf16(p2, p3);
          }
          tc::tmem_st16(s_addr + cc * 16, pk);
        }
      }
      if (moved) l *= alpha;
      l += (sum01.x + sum01.y) + (sum23.x + sum23.y);
      tc::tmem_st_wait();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(B_PFULL + sbuf));
    }
    if (ok && n_kvw > 0) ok = tc::mbar_wait(bar(B_PVDONE + w), (n_kvw - 1) & 1, status, 210);
    tc::tc_fence_after();
    if (ok && n_kvw > 0) {
      const bool live = gi < P.seq;
      const float inv = live ? 1.f / l : 0.f;
#pragma unroll
      for (int cc = 0; cc < HD / 32; ++cc) {
        uint32_t o[32];
        tc::tmem_ld32(o_addr + cc * 32, o);
        tc::tmem_ld_wait();
        if (gi < P.t_pad) {
          const int col = h * HD + cc * 32;
          __nv_bfloat16* dst = P.a + ((long long)(col / 64) * P.n_pad + row0 + gi) * 64 + (col % 64);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            uint4 v;
            v.x = tc::pack_bf16(__uint_as_float(o[k * 8 + 0]) * inv, __uint_as_float(o[k * 8 + 1]) * inv);
            v.y = tc::pack_bf16(__uint_as_float(o[k * 8 + 2]) * inv, __uint_as_float(o[k * 8 + 3]) * inv);
            v.z = tc::pack_bf16(__uint_as_float(o[k * 8 + 4]) * inv, __uint_as_float(o[k * 8 + 5]) * inv);
            v.w = tc::pack_bf16(__uint_as_float(o[k * 8 + 6]) * inv, __uint_as_float(o[k * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + 8 * k) = v;
          }
        }
      }
      if (gi < P.t_pad) P.lse[((long long)b * P.hq + h) * P.t_pad + gi] = live ? m * P.scale + logf(l) : 0.f;
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

template <int HD, int TILES>
cudaError_t fwd_launch_t(const fbl_plan* p, AttnFwdParams& P, int n_qt, cudaStream_t st) {
  auto k = attn_fwd_tc_kernel<HD, TILES>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FwdSmem<HD, TILES>::TOTAL);
  if (e != cudaSuccess) return e;
  if (TILES == 1) P.pair = 0;
  P.batch = p->d.batch;
  P.n_slots = P.pair ? (n_qt + 1) / 2 : n_qt;
  P.chunk = chunk_for((long long)p->seq_kv * HD * 4, p->d.n_q_heads * p->d.batch, 96ll << 20);   // K and V of one head
  dim3 grid((unsigned)(P.n_slots * p->d.n_q_heads * p->d.batch));
  return launch_pdl(k, grid, dim3(64 + 128 * TILES), FwdSmem<HD, TILES>::TOTAL, st, P);
}

template <int HD>
cudaError_t fwd_launch(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                       int32_t* status, cudaStream_t st) {
  AttnFwdParams P;
  memset(&P, 0, sizeof(P));
  const int panels = HD / 64;
  if (!fbl_encode_rtile_map(&P.tq, Q, p->n_pad, p->dq / 64, BQ, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tk, K, p->n_pad_kv, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tv, V, p->n_pad_kv, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  P.a = (__nv_bfloat16*)A; P.lse = lse; P.n_pad = p->n_pad;
  P.seq = p->d.seq; P.t_pad = p->t_pad; P.hq = p->d.n_q_heads; P.group = p->group; P.causal = p->d.causal;
  P.seq_k = p->seq_kv; P.t_pad_k = p->t_pad_kv;
  P.scale = p->scale; P.status = status;
  const int n_qt = (p->d.seq + BQ - 1) / BQ;
  // two query tiles per block when that still leaves at least one block per SM
  P.pair = (n_qt >= 2 && (long long)((n_qt + 1) / 2) * p->d.n_q_heads * p->d.batch >= p->sm_count) ? 1 : 0;
  if (HD == 64) {
    // tuning knob: 1 = one query tile per block and two blocks per SM, 2 = two tiles per block; default by sequence length
    const int mode = p->knob_fwd_tiles;
    if (mode == 1 || (mode == 0 && n_qt <= 4)) return fwd_launch_t<64, 1>(p, P, n_qt, st);
  }
  return fwd_launch_t<HD, 2>(p, P, n_qt, st);
}

// ---------------------------------------------------------------------------------------------------
// Backward: one block per (128-key tile, KV head, batch).  For every query head of the group and every
// query tile it recomputes the transposed scores S^T = K Q^T and dP^T = V dO^T on the tensor pipe (so
// the rows a thread owns are keys), forms P^T = exp(S^T - LSE) and dS^T = P^T * (dP^T - D) in registers,
// and writes both once to swizzled shared memory.  Those two tiles then feed three products:
//   dV += P^T dO  and  dK += dS^T Q   (sequence-axis reductions; accumulators stay in TMEM over the
//                                      whole query loop and over the G heads of the group), and
//   dQ  = dS K    (the same dS^T bytes read MN-major, i.e. transposed by descriptor), a key-axis
//                  reduction across blocks, added to an fp32 buffer with vector red operations.
// ---------------------------------------------------------------------------------------------------
struct alignas(64) AttnBwdParams {
  CUtensorMap tq, tk, tv, tdo, tdq;   // tdq: fp32 dQ accumulator, target of the bulk reductions
  const float* lse;      // [B, Hq, t_pad]
  const float* dvec;     // [B, Hq, t_pad]   D = rowsum(dO * O)
  float* dqacc;          // fp32 [n_pad, dq] in the bf16 tile order
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  long long n_pad, n_pad_k;          // rows of the query-side (Q, dO, dQ) and key-side (K, V, dK, dV) buffers
  int seq, t_pad, hq, group, causal, dkv;
  int seq_k, t_pad_k;                // key-side sequence length and padded length
  int batch, chunk;      // grid = key tiles * KV heads * batch blocks, see decode_block
  float scale;
  int32_t* status;
};

// P^T never touches shared memory: the softmax warps store it (bf16, two per column) over the S^T columns
// in tensor memory once every warp has read them, and dV += P^T dO takes its A operand from there.  HD = 64
// has spare TMEM columns for dQ and shared memory to double-buffer Q/dO and dS^T, so the tensor pipe computes
// the next tile's S^T / dP^T and this tile's dK, dQ while the softmax warps are busy.  HD = 128 fills TMEM
// (S^T, dP^T, dV, dK = 512 columns): dQ reuses the dP^T columns, so only the next S^T can be issued before dQ
// has been drained.  Both keep a separate staging area for the asynchronous dQ reduction.
template <int HD>
struct BwdSmem {
  static constexpr bool PIPE = HD == 64;
  // stages: Q (needed first, for the next S^T, and freed last, by dK) three deep, dO and dS^T two deep, one dQ
  // staging tile; everything single at HD = 128
  static constexpr uint32_t NQQ = PIPE ? 3 : 1, NDO = PIPE ? 2 : 1, NP = PIPE ? 2 : 1, NS = 1;
  static constexpr uint32_t PANELS = HD / 64;
  static constexpr uint32_t TILE = PANELS * 16384;
  static constexpr uint32_t STAGE_BYTES = 128 * HD * 4;               // one fp32 dQ tile
  static constexpr uint32_t K_OFF = 0, V_OFF = TILE, Q_OFF = 2 * TILE, DO_OFF = Q_OFF + NQQ * TILE;
  static constexpr uint32_t DS_OFF = DO_OFF + NDO * TILE, STAGE_OFF = DS_OFF + NP * 32768;
  static constexpr uint32_t LSE_OFF = STAGE_OFF + NS * STAGE_BYTES;    // 128 floats of LSE per Q stage, then 128 of D per dO stage
  static constexpr uint32_t D_OFF = LSE_OFF + NQQ * 512;
  static constexpr uint32_t BAR_OFF = D_OFF + NDO * 512;
  static constexpr uint32_t N_BARS = 24;          // BB_* below: 22 in use
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16;
};

enum { BB_KVFULL = 0, BB_QFULL = 1, BB_QEMPTY = 4, BB_DOFULL = 7, BB_DOEMPTY = 9, BB_SFULL = 11, BB_PDSFULL, BB_DQFULL, BB_DQDRAINED, BB_DQSTAGED, BB_STAGEFREE = BB_DQSTAGED + 2, BB_SREAD = BB_STAGEFREE + 2, BB_DVDONE, BB_DPFULL };

constexpr int BWD_THREADS = 608;     // warp 0 TMA loads, warp 1 MMA, warps 2-17 softmax (four per TMEM lane quarter), warp 18 dQ reductions
constexpr int BWD_SM_THREADS = 512;

template <int HD>
__global__ void __launch_bounds__(BWD_THREADS, 1) attn_bwd_tc_kernel(const __grid_constant__ AttnBwdParams P) {
  using SM = BwdSmem<HD>;
  constexpr bool PIPE = SM::PIPE;
  constexpr uint32_t PANELS = SM::PANELS, NQQ = SM::NQQ, NDO = SM::NDO, NP = SM::NP, NS = SM::NS;
  constexpr uint32_t S_COL = 0, DP_COL = 128, DV_COL = 256, DK_COL = 256 + HD;
  constexpr uint32_t DQ_COL = PIPE ? 384 : DP_COL;   // HD = 128: dQ reuses the dP^T columns
  constexpr uint32_t P_COL = PIPE ? 448 : S_COL;     // HD = 64: own columns; HD = 128: P^T overwrites S^T in place
  constexpr uint32_t TMEM_COLS = 512;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = tc::smem_u32(smem_raw);
  const uint32_t bars = base + SM::BAR_OFF;
  const uint32_t slot = bars + 8 * SM::N_BARS;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  // under a causal mask key tile 0 has the most query tiles: it is slot 0
  const int n_kvh = P.hq / P.group;
  int slot_i, gb;
  decode_block((int)blockIdx.x, (P.t_pad_k + BKV - 1) / BKV, n_kvh * P.batch, P.chunk, &slot_i, &gb);
  const int j0 = slot_i * BKV, g = gb % n_kvh, b = gb / n_kvh;
  const int row0 = b * P.t_pad, row0k = b * P.t_pad_k;
  const int n_qt = (P.seq + BQ - 1) / BQ;
  const int qt_begin = P.causal ? j0 / BQ : 0;
  const int per_head = n_qt - qt_begin;
  const int n_it = P.group * per_head;
  int32_t* status = P.status;
  if ((base & 1023u) != 0) {                    // the swizzled tiles need a 1024-byte aligned window
    if (threadIdx.x == 0) atomicCAS(status, 0, 399);
    return;
  }

  if (threadIdx.x == 0) {
    tc::mbar_init(bar(BB_KVFULL), 1);
    for (int s = 0; s < 3; ++s) {
      tc::mbar_init(bar(BB_QFULL + s), 1);
      tc::mbar_init(bar(BB_QEMPTY + s), 1);
    }
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(bar(BB_DOFULL + s), 1);
      tc::mbar_init(bar(BB_DOEMPTY + s), 1);
    }
    tc::mbar_init(bar(BB_SFULL), 1);
    tc::mbar_init(bar(BB_PDSFULL), BWD_SM_THREADS);
    tc::mbar_init(bar(BB_DQFULL), 1);
    tc::mbar_init(bar(BB_DQDRAINED), BWD_SM_THREADS);
    tc::mbar_init(bar(BB_DQSTAGED), BWD_SM_THREADS);
    tc::mbar_init(bar(BB_DQSTAGED + 1), BWD_SM_THREADS);
    tc::mbar_init(bar(BB_STAGEFREE), 1);
    tc::mbar_init(bar(BB_STAGEFREE + 1), 1);
    tc::mbar_init(bar(BB_SREAD), BWD_SM_THREADS);
    tc::mbar_init(bar(BB_DVDONE), 1);
    tc::mbar_init(bar(BB_DPFULL), 1);
    tc::fence_barrier_init();
    // This thread is the TMA producer: K, V and the first Q tile (forward-pass data) are requested right here, so
    // that their latency overlaps the tensor-memory allocation and the block-wide barrier below.
    tc::tma_prefetch_desc(&P.tk); tc::tma_prefetch_desc(&P.tv); tc::tma_prefetch_desc(&P.tq);
    tc::tma_prefetch_desc(&P.tdo); tc::tma_prefetch_desc(&P.tdq);
    tc::mbar_expect_tx(bar(BB_KVFULL), 2 * SM::TILE);
    tc::tma_load_3d(base + SM::K_OFF, &P.tk, bar(BB_KVFULL), 0, row0k + j0, g * (int)PANELS);
    tc::tma_load_3d(base + SM::V_OFF, &P.tv, bar(BB_KVFULL), 0, row0k + j0, g * (int)PANELS);
    if (n_it > 0) {
      // LSE travels with Q and D with dO: 128 floats each, into the iteration's staging buffer
      tc::mbar_expect_tx(bar(BB_QFULL), SM::TILE + 512);
      tc::tma_load_3d(base + SM::Q_OFF, &P.tq, bar(BB_QFULL), 0, row0 + qt_begin * BQ, g * P.group * (int)PANELS);
      tc::bulk_load(base + SM::LSE_OFF, P.lse + ((long long)b * P.hq + g * P.group) * P.t_pad + qt_begin * BQ, 512, bar(BB_QFULL));
    }
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
  // Where a block's dQ tiles are staged for the bulk reduction: one staging tile; with the pipelined variant the
  // last tile goes to the dS^T buffer that the last iteration does not use (its readers, the dK and dQ products of
  // the tile before, are complete by then), so the block's final drain does not wait for the previous reduction.
  auto stage_is_alt = [&](int dit) { return PIPE && dit == n_it - 1 && n_it >= 2; };
  auto stage_addr = [&](int dit) -> uint32_t {
    return stage_is_alt(dit) ? base + SM::DS_OFF + (uint32_t)(n_it % (int)NP) * 32768u
                             : base + SM::STAGE_OFF + (uint32_t)(dit % (int)NS) * SM::STAGE_BYTES;
  };
  // Of this kernel's inputs only dO (and D) come from the kernel before it (the dA GEMM); K, V, Q and LSE are the
  // forward pass's.  Each role therefore waits for that kernel where it first needs it: the producer has K, V
  // and the first Q tile on their way before it does.
  if (warp == 0 && lane == 0) {
    // ---- TMA producer ------------------------------------------------------------------------
    // (K, V and Q of the first tile were requested during set-up)
    bool waited = false;
    for (int it = 0; it < n_it; ++it) {
      const int h = g * P.group + it / per_head, qt = qt_begin + it % per_head;
      // LSE travels with Q and D with dO, 128 floats each.  A stage's previous readers (the products, and for
      // LSE / D the softmax warps, which finish a tile before its dK and dV products are issued) are behind the
      // barrier that frees it.  Rows past the sequence end may hold anything: the softmax warps mask them.
      const long long stat_off = ((long long)b * P.hq + h) * P.t_pad + qt * BQ;
      const uint32_t sq = it % NQQ, sd = it % NDO;
      if (it > 0) {
        if (!tc::mbar_wait(bar(BB_QEMPTY + sq), ((it / NQQ) & 1) ^ 1, status, 301)) break;
        tc::mbar_expect_tx(bar(BB_QFULL + sq), SM::TILE + 512);
        tc::tma_load_3d(base + SM::Q_OFF + sq * SM::TILE, &P.tq, bar(BB_QFULL + sq), 0, row0 + qt * BQ, h * (int)PANELS);
        tc::bulk_load(base + SM::LSE_OFF + sq * 512, P.lse + stat_off, 512, bar(BB_QFULL + sq));
      }
      if (!tc::mbar_wait(bar(BB_DOEMPTY + sd), ((it / NDO) & 1) ^ 1, status, 313)) break;
      if (!waited) { pdl_wait(); waited = true; }
      tc::mbar_expect_tx(bar(BB_DOFULL + sd), SM::TILE + 512);
      tc::tma_load_3d(base + SM::DO_OFF + sd * SM::TILE, &P.tdo, bar(BB_DOFULL + sd), 0, row0 + qt * BQ, h * (int)PANELS);
      tc::bulk_load(base + SM::D_OFF + sd * 512, P.dvec + stat_off, 512, bar(BB_DOFULL + sd));
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer --------------------------------------------------------------------------
    const uint32_t idesc_s = tc::idesc_bf16(BKV, BQ, 0, 0);
    const uint32_t idesc_kv = tc::idesc_bf16(BKV, HD, 0, 1);
    const uint32_t idesc_dq = tc::idesc_bf16(BQ, HD, 1, 1);
    // Descriptor words are formed once; per instruction only the start-address field of the low word moves
    // (offsets below are in 16-byte units: a 64-column panel is 1024, a 16-element step along a row 2, 16 rows 128).
    const uint32_t hi = tc::smem_desc_hi(1024);
    const uint32_t k_km = tc::smem_desc_lo(base + SM::K_OFF, 16), k_mn = tc::smem_desc_lo(base + SM::K_OFF, 16384);
    const uint32_t v_km = tc::smem_desc_lo(base + SM::V_OFF, 16);
    const uint32_t q_km = tc::smem_desc_lo(base + SM::Q_OFF, 16), q_mn = tc::smem_desc_lo(base + SM::Q_OFF, 16384);
    const uint32_t do_km = tc::smem_desc_lo(base + SM::DO_OFF, 16), do_mn = tc::smem_desc_lo(base + SM::DO_OFF, 16384);
    const uint32_t ds_km = tc::smem_desc_lo(base + SM::DS_OFF, 16), ds_mn = tc::smem_desc_lo(base + SM::DS_OFF, 16384);
    auto issue_s = [&](int it) {              // S^T = K Q^T of tile `it`
      const uint32_t qs = q_km + (it % NQQ) * (SM::TILE >> 4);
#pragma unroll
      for (uint32_t kk = 0; kk < HD / 16; ++kk) {
        const uint32_t o = (kk / 4) * 1024 + (kk % 4) * 2;
        tc::mma_bf16_ss_w(tmem_base + S_COL, k_km + o, hi, qs + o, hi, idesc_s, kk > 0);
      }
      if (!PIPE) tc::mma_commit(bar(BB_SFULL));     // HD = 128: the softmax warps start on the scores while dP^T is
    };                                              // still to come (it waits for the previous tile's dQ drain)
    auto issue_dp = [&](int it) {             // dP^T = V dO^T of tile `it`, announced on its own barrier
      const uint32_t dos = do_km + (it % NDO) * (SM::TILE >> 4);
#pragma unroll
      for (uint32_t kk = 0; kk < HD / 16; ++kk) {
        const uint32_t o = (kk / 4) * 1024 + (kk % 4) * 2;
        tc::mma_bf16_ss_w(tmem_base + DP_COL, v_km + o, hi, dos + o, hi, idesc_s, kk > 0);
      }
      tc::mma_commit(bar(PIPE ? BB_SFULL : BB_DPFULL));      // HD = 64: one announcement for both score tiles
    };
    auto issue_dv = [&](int it) {             // dV += P^T dO, P^T read from tensor memory
      const uint32_t dos = do_mn + (it % NDO) * (SM::TILE >> 4);
#pragma unroll
      for (uint32_t kk = 0; kk < BQ / 16; ++kk)                      // dO: MN-major, 16 query rows per step;
        tc::mma_bf16_ts_w(tmem_base + DV_COL, tmem_base + P_COL + kk * 8,   // 16 queries = 8 packed columns
                          dos + kk * 128, hi, idesc_kv, (it > 0 || kk > 0) ? 1u : 0u);
    };
    auto issue_dk = [&](int it) {             // dK += dS^T Q
      const uint32_t qs = q_mn + (it % NQQ) * (SM::TILE >> 4);
      const uint32_t dss = ds_km + (it % NP) * 2048;
#pragma unroll
      for (uint32_t kk = 0; kk < BQ / 16; ++kk) {
        const uint32_t ao = (kk / 4) * 1024 + (kk % 4) * 2;        // dS^T: K-major, reduction over queries
        tc::mma_bf16_ss_w(tmem_base + DK_COL, dss + ao, hi, qs + kk * 128, hi, idesc_kv,   // Q: MN-major, 16 query rows
                          (it > 0 || kk > 0) ? 1u : 0u);
      }
    };
    auto issue_dq = [&](int it) {             // dQ = dS K: the dS^T tile read MN-major, i.e. transposed by descriptor
      const uint32_t dss = ds_mn + (it % NP) * 2048;
#pragma unroll
      for (uint32_t kk = 0; kk < BKV / 16; ++kk)                     // both operands MN-major: 16 key rows per step
        tc::mma_bf16_ss_w(tmem_base + DQ_COL, dss + kk * 128, hi, k_mn + kk * 128, hi, idesc_dq, kk > 0);
      tc::mma_commit(bar(BB_DQFULL));
    };
    bool ok = tc::mbar_wait(bar(BB_KVFULL), 0, status, 302);
    if (ok && n_it > 0) {
      ok = tc::mbar_wait(bar(BB_QFULL), 0, status, 303) && tc::mbar_wait(bar(BB_DOFULL), 0, status, 314);
      if (ok) { tc::tc_fence_after(); issue_s(0); issue_dp(0); }
    }
    if (PIPE) {
      // P^T has its own columns here, so the next tile's products come first and the softmax warps start on
      // tile it + 1 while the tensor pipe works on dV, dK, dQ of tile it
      for (int it = 0; it < n_it && ok; ++it) {
        if (it + 1 < n_it) {
          // S^T(it+1) as soon as every softmax warp has copied S^T(it) to registers: it is computed while
          // they work on tile it
          if (!tc::mbar_wait(bar(BB_SREAD), it & 1, status, 311)) { ok = false; break; }
          if (!tc::mbar_wait(bar(BB_QFULL + ((it + 1) % NQQ)), ((it + 1) / NQQ) & 1, status, 303)) { ok = false; break; }
          tc::tc_fence_after();
          issue_s(it + 1);
        }
        if (!tc::mbar_wait(bar(BB_PDSFULL), it & 1, status, 305)) { ok = false; break; }
        tc::tc_fence_after();
        if (it + 1 < n_it) {
          if (!tc::mbar_wait(bar(BB_DOFULL + ((it + 1) % NDO)), ((it + 1) / NDO) & 1, status, 314)) { ok = false; break; }
          issue_dp(it + 1);                             // dP^T(it) has been read as well: announce tile it + 1
        }
        issue_dv(it);
        tc::mma_commit(bar(BB_DVDONE));                 // P^T(it) has been read: P^T(it+1) may be stored
        tc::mma_commit(bar(BB_DOEMPTY + (it % NDO)));   // ... and dO of this tile is not read again
        issue_dk(it);
        tc::mma_commit(bar(BB_QEMPTY + (it % NQQ)));    // nor is Q
        if (it > 0 && !tc::mbar_wait(bar(BB_DQDRAINED), (it - 1) & 1, status, 304)) { ok = false; break; }
        tc::tc_fence_after();
        issue_dq(it);
      }
    } else {
      for (int it = 0; it < n_it && ok; ++it) {
        if (!tc::mbar_wait(bar(BB_PDSFULL), it & 1, status, 305)) { ok = false; break; }
        tc::tc_fence_after();
        // dQ first: its drain to shared memory (which frees the dP^T columns for the next tile) then overlaps
        // the dV and dK products
        issue_dq(it);
        issue_dk(it);
        tc::mma_commit(bar(BB_QEMPTY));                 // Q of this tile is not read again: the next one is fetched
        issue_dv(it);                                   // while dV runs
        tc::mma_commit(bar(BB_DOEMPTY));                // ... and dO
        if (it + 1 < n_it) {
          if (!tc::mbar_wait(bar(BB_QFULL), (it + 1) & 1, status, 303)) { ok = false; break; }
          tc::tc_fence_after();
          issue_s(it + 1);                   // the S^T columns (P^T by now) were last read by dV above
          if (!tc::mbar_wait(bar(BB_DQDRAINED), it & 1, status, 304)) { ok = false; break; }
          if (!tc::mbar_wait(bar(BB_DOFULL), (it + 1) & 1, status, 314)) { ok = false; break; }
          tc::tc_fence_after();
          issue_dp(it + 1);                  // the dP^T columns held dQ until it was drained
        }
      }
      // dQ is issued first here, so its barrier does not cover the last tile's dK and dV products: one more
      // arrival, on the barrier the pipelined variant uses for dV, tells the epilogue that they are complete
      if (ok && n_it > 0) tc::mma_commit(bar(BB_DVDONE));
    }
  } else if (warp == 18) {
    // ---- dQ reduction warp: adds each staged dQ tile to the fp32 accumulator with bulk tensor reductions ----
    if (lane == 0) {
      pdl_wait();                                    // the accumulator's zero-fill precedes the kernel before this one
      for (int dit = 0; dit < n_it; ++dit) {
        const int h = g * P.group + dit / per_head, i0 = (qt_begin + dit % per_head) * BQ;
        if (!tc::mbar_wait(bar(BB_DQSTAGED + (dit % NS)), (dit / (int)NS) & 1, status, 309)) break;   // one per buffer, like STAGEFREE
        const uint32_t stage = stage_addr(dit);
#pragma unroll
        for (int pn = 0; pn < (int)PANELS; ++pn)
          tc::tma_reduce_add_4d(&P.tdq, stage + pn * 32768, 0, 0, row0 + i0, h * (int)PANELS + pn);
        tc::bulk_commit_group();
        tc::bulk_wait_group_read0();                 // the staging tile has been read: it may be overwritten
        tc::mbar_arrive(bar(BB_STAGEFREE + (dit % NS)));     // one barrier per staging buffer: a waiter is never
                                                             // more than one phase behind
      }
      tc::bulk_wait_group0();
    }
  } else if (warp >= 2) {
    // ---- softmax warps: thread = (key row, one quarter of the 128 query columns) -----------------------
    const int q = warp % 4;                         // TMEM lane quarter
    const int part = (warp - 2) / 4;                // which 32 query columns (and which quarter of HD later)
    const int r = q * 32 + lane;
    const int t = threadIdx.x - 64;                 // 0..511
    const int gj = j0 + r;
    pdl_wait();                                     // D is written by the kernel before this one; dK, dV may still be read by it
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const float c = P.scale * LOG2E;
    float* s_stage = reinterpret_cast<float*>(smem_raw + SM::LSE_OFF);
    bool ok = true;

    // dQ tile of iteration `dit` (row = query i0 + row): each thread copies its TMEM row segment, scaled, to a
    // staging tile in shared memory in the 128-byte-swizzled box layout of the accumulator's tensor map; the
    // reduction warp then adds the whole tile to global memory asynchronously, off the critical path.
    auto drain_dq = [&](int dit) -> bool {
      const uint32_t stage = stage_addr(dit);
      if (!tc::mbar_wait(bar(BB_DQFULL), dit & 1, status, 307)) return false;
      tc::tc_fence_after();
      // this thread's HD / 4 accumulator columns in one go; the tensor pipe gets the columns back (at HD = 128 the
      // next tile's dP^T waits for them) as soon as they are in registers, before the stores to the staging tile
      constexpr int NC = HD / 4;                     // 16 or 32 columns
      const int c0 = part * NC;
      uint32_t o[NC];
      if constexpr (NC == 32) tc::tmem_ld32(lane_addr + DQ_COL + c0, o);
      else tc::tmem_ld16(lane_addr + DQ_COL + c0, o);
      tc::tmem_ld_wait();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(BB_DQDRAINED));            // TMEM side done: the tensor pipe may reuse the columns
      // Only now wait for the staging buffer (its previous tile must have been read by its bulk reduction, which
      // takes a few thousand cycles): the values sit in registers meanwhile and the columns are already free.
      if (dit >= (int)NS && !stage_is_alt(dit) && !tc::mbar_wait(bar(BB_STAGEFREE + (dit % NS)), (dit / (int)NS - 1) & 1, status, 310)) return false;
#pragma unroll
      for (int u = 0; u < NC / 16; ++u) {            // 16 columns = half of a 128-byte unit of the box
        const int cu = c0 + u * 16;
        const uint32_t unit = (uint32_t)(r * 2 + (cu % 64) / 32);
        const uint32_t rowaddr = stage + (cu / 64) * 32768 + unit * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t chk = (uint32_t)((cu % 32) / 4 + k);
          const uint32_t addr = rowaddr + ((chk ^ (unit & 7)) * 16);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(__uint_as_float(o[u * 16 + 4 * k]) * P.scale),
                       "f"(__uint_as_float(o[u * 16 + 4 * k + 1]) * P.scale), "f"(__uint_as_float(o[u * 16 + 4 * k + 2]) * P.scale),
                       "f"(__uint_as_float(o[u * 16 + 4 * k + 3]) * P.scale) : "memory");
        }
      }
      tc::fence_proxy_async();
      tc::mbar_arrive(bar(BB_DQSTAGED + (dit % NS)));     // staging side done: the reduction warp takes over
      return true;
    };

    int c_q = 0;                                    // query tile within the head of the tile being processed
    for (int it = 0; it < n_it && ok; ++it) {
      const int i0 = (qt_begin + c_q) * BQ;
      if (++c_q == per_head) c_q = 0;
      // LSE and D of this query tile were copied to shared memory by the producer (a buffer per Q / dO stage)
      // and arrived before the score products awaited below were issued
      const float* s_lse = s_stage + (it % NQQ) * 128;
      const float* s_d = s_stage + NQQ * 128 + (it % NDO) * 128;
      if (!tc::mbar_wait(bar(BB_SFULL), it & 1, status, 306)) { ok = false; break; }
      tc::tc_fence_after();
      // element masks are needed only on the diagonal tile and on tiles with keys or queries beyond the sequence
      const bool need_mask = (P.causal && (i0 < j0 + BKV - 1)) || (j0 + BKV > P.seq_k) || (i0 + BQ > P.seq);
      const uint32_t dsrow = base + SM::DS_OFF + (it % NP) * 32768 + (part / 2) * 16384 + r * 128;
      // this thread's 32 score columns first: with HD = 128 the packed P^T overwrites S^T columns that belong to
      // other warps of the same lane quarter, so every warp must have read its scores before any P^T store
      uint32_t sv[32];
      tc::tmem_ld32(lane_addr + S_COL + part * 32, sv);
      tc::tmem_ld_wait();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(BB_SREAD));                   // this thread's scores are in registers
      if (!PIPE) {
        if (!tc::mbar_wait(bar(BB_SREAD), it & 1, status, 311)) { ok = false; break; }
        tc::tc_fence_after();
      }
      if constexpr (PIPE) {
      // One 16-column chunk: P^T = exp2(S^T c - LSE) to tensor memory, dS^T = P^T (dP^T - D) to the swizzled
      // shared-memory operand tile, both rounded to bf16.  MASKED is the rare path (diagonal / ragged tiles).
      auto chunk = [&](int cc, auto masked_tag) {
        constexpr bool MASKED = decltype(masked_tag)::value;
        const int c0 = part * 32 + cc * 16;
        uint32_t dpv[16];
        tc::tmem_ld16(lane_addr + DP_COL + c0, dpv);
        tc::tmem_ld_wait();
        uint32_t pp[8], dd[8];
#pragma unroll
        for (int k = 0; k < 16; k += 4) {
          const float4 l4 = *reinterpret_cast<const float4*>(&s_lse[c0 + k]);
          const float4 d4 = *reinterpret_cast<const float4*>(&s_d[c0 + k]);
          // two-wide fp32 operations (one instruction per pair): x = S^T c - LSE log2e, then dS^T = P^T (dP^T - D)
          const float2 c2 = make_float2(c, c);
          const float2 nl2e = make_float2(-LOG2E, -LOG2E), neg1 = make_float2(-1.f, -1.f);
          const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(sv[cc * 16 + k]), __uint_as_float(sv[cc * 16 + k + 1])), c2, __fmul2_rn(make_float2(l4.x, l4.y), nl2e));
          const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(sv[cc * 16 + k + 2]), __uint_as_float(sv[cc * 16 + k + 3])), c2, __fmul2_rn(make_float2(l4.z, l4.w), nl2e));
          float pv[4] = {tc::fast_exp2(x01.x), tc::fast_exp2(x01.y), tc::fast_exp2(x23.x), tc::fast_exp2(x23.y)};
          if (MASKED) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int gi = i0 + c0 + k + u;
              if (gj >= P.seq_k || gi >= P.seq || (P.causal && gi < gj)) pv[u] = 0.f;
            }
          }
          const float2 g01 = __fmul2_rn(make_float2(pv[0], pv[1]), __ffma2_rn(make_float2(d4.x, d4.y), neg1, make_float2(__uint_as_float(dpv[k]), __uint_as_float(dpv[k + 1]))));
          const float2 g23 = __fmul2_rn(make_float2(pv[2], pv[3]), __ffma2_rn(make_float2(d4.z, d4.w), neg1, make_float2(__uint_as_float(dpv[k + 2]), __uint_as_float(dpv[k + 3]))));
          float gv[4] = {g01.x, g01.y, g23.x, g23.y};
          if (MASKED) {                              // LSE / D of rows past the sequence end are not defined
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int gi = i0 + c0 + k + u;
              if (gj >= P.seq_k || gi >= P.seq || (P.causal && gi < gj)) gv[u] = 0.f;
            }
          }
          pp[k / 2] = tc::pack_bf16(pv[0], pv[1]);
          pp[k / 2 + 1] = tc::pack_bf16(pv[2], pv[3]);
          dd[k / 2] = tc::pack_bf16(gv[0], gv[1]);
          dd[k / 2 + 1] = tc::pack_bf16(gv[2], gv[3]);
        }
        if (PIPE && cc == 0 && it > 0) {
          // P^T has its own columns, single-buffered: the dV product of the previous tile must have read them.
          // The wait sits here, behind the first chunk's arithmetic, which needs only S^T and dP^T.
          if (!tc::mbar_wait(bar(BB_DVDONE), (it - 1) & 1, status, 312)) { ok = false; return; }
          tc::tc_fence_after();
        }
        tc::tmem_st8(lane_addr + P_COL + c0 / 2, pp);
        // 16 query columns = 2 swizzled 16-byte chunks of this key row inside its 64-query panel
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          const uint32_t chk = (uint32_t)((part % 2) * 4 + cc * 2 + ch);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dsrow + ((chk ^ (uint32_t)(r & 7)) * 16)),
                       "r"(dd[ch * 4]), "r"(dd[ch * 4 + 1]), "r"(dd[ch * 4 + 2]), "r"(dd[ch * 4 + 3]) : "memory");
        }
      };
      if (need_mask) {
        chunk(0, std::true_type{});
        if (ok) chunk(1, std::true_type{});
      } else {
        chunk(0, std::false_type{});
        if (ok) chunk(1, std::false_type{});
      }
      } else {
      // Phase A needs only S^T: P^T = exp2(S^T c - LSE) for this thread's 32 query columns, kept in the score
      // registers as fp32 and stored to tensor memory as bf16.  It runs while the tensor pipe is still busy with
      // dP^T of this tile (which at HD = 128 also waits for the previous tile's dQ to be drained).
      auto phase_a = [&](auto masked_tag) {
        constexpr bool MASKED = decltype(masked_tag)::value;
        const float2 c2 = make_float2(c, c), nl2e = make_float2(-LOG2E, -LOG2E);
#pragma unroll
        for (int k = 0; k < 32; k += 4) {
          const float4 l4 = *reinterpret_cast<const float4*>(&s_lse[part * 32 + k]);
          const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(sv[k]), __uint_as_float(sv[k + 1])), c2, __fmul2_rn(make_float2(l4.x, l4.y), nl2e));
          const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(sv[k + 2]), __uint_as_float(sv[k + 3])), c2, __fmul2_rn(make_float2(l4.z, l4.w), nl2e));
          float pv[4] = {tc::fast_exp2(x01.x), tc::fast_exp2(x01.y), tc::fast_exp2(x23.x), tc::fast_exp2(x23.y)};
          if (MASKED) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int gi = i0 + part * 32 + k + u;
              if (gj >= P.seq_k || gi >= P.seq || (P.causal && gi < gj)) pv[u] = 0.f;
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) sv[k + u] = __float_as_uint(pv[u]);
        }
      };
      if (need_mask) phase_a(std::true_type{}); else phase_a(std::false_type{});
      {
        uint32_t pp[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) pp[k] = tc::pack_bf16(__uint_as_float(sv[2 * k]), __uint_as_float(sv[2 * k + 1]));
        if (PIPE && it > 0) {
          // P^T has its own columns, single-buffered: the dV product of the previous tile must have read them
          if (!tc::mbar_wait(bar(BB_DVDONE), (it - 1) & 1, status, 312)) { ok = false; break; }
          tc::tc_fence_after();
        }
        tc::tmem_st16(lane_addr + P_COL + part * 16, pp);
      }
      // Phase B: dS^T = P^T (dP^T - D), rounded to bf16, to the swizzled shared-memory operand tile, in two
      // 16-column chunks.  MASKED is the rare path (diagonal / ragged tiles).
      if (!tc::mbar_wait(bar(BB_DPFULL), it & 1, status, 316)) { ok = false; break; }
      tc::tc_fence_after();
      auto phase_b = [&](int cc, auto masked_tag) {
        constexpr bool MASKED = decltype(masked_tag)::value;
        const int c0 = part * 32 + cc * 16;
        uint32_t dpv[16];
        tc::tmem_ld16(lane_addr + DP_COL + c0, dpv);
        tc::tmem_ld_wait();
        uint32_t dd[8];
        const float2 neg1 = make_float2(-1.f, -1.f);
#pragma unroll
        for (int k = 0; k < 16; k += 4) {
          const float4 d4 = *reinterpret_cast<const float4*>(&s_d[c0 + k]);
          const float* pv = reinterpret_cast<const float*>(&sv[cc * 16 + k]);
          const float2 g01 = __fmul2_rn(make_float2(pv[0], pv[1]), __ffma2_rn(make_float2(d4.x, d4.y), neg1, make_float2(__uint_as_float(dpv[k]), __uint_as_float(dpv[k + 1]))));
          const float2 g23 = __fmul2_rn(make_float2(pv[2], pv[3]), __ffma2_rn(make_float2(d4.z, d4.w), neg1, make_float2(__uint_as_float(dpv[k + 2]), __uint_as_float(dpv[k + 3]))));
          float gv[4] = {g01.x, g01.y, g23.x, g23.y};
          if (MASKED) {                              // LSE / D of rows past the sequence end are not defined
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const int gi = i0 + c0 + k + u;
              if (gj >= P.seq_k || gi >= P.seq || (P.causal && gi < gj)) gv[u] = 0.f;
            }
          }
          dd[k / 2] = tc::pack_bf16(gv[0], gv[1]);
          dd[k / 2 + 1] = tc::pack_bf16(gv[2], gv[3]);
        }
        // 16 query columns = 2 swizzled 16-byte chunks of this key row inside its 64-query panel
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          const uint32_t chk = (uint32_t)((part % 2) * 4 + cc * 2 + ch);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dsrow + ((chk ^ (uint32_t)(r & 7)) * 16)),
                       "r"(dd[ch * 4]), "r"(dd[ch * 4 + 1]), "r"(dd[ch * 4 + 2]), "r"(dd[ch * 4 + 3]) : "memory");
        }
      };
      if (need_mask) { phase_b(0, std::true_type{}); phase_b(1, std::true_type{}); }
      else { phase_b(0, std::false_type{}); phase_b(1, std::false_type{}); }
      }
      if (!ok) break;
      tc::tmem_st_wait();
      tc::fence_proxy_async();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(BB_PDSFULL));
      if (PIPE) {
        if (it > 0) ok = drain_dq(it - 1);
      } else {
        ok = drain_dq(it);
      }
    }
    if (PIPE && ok && n_it > 0) ok = drain_dq(n_it - 1);
    // dK, dV of this key tile: every MMA has completed (HD = 64: dQ is the last product issued, and the wait for
    // it is behind us; HD = 128: the extra arrival above)
    if (!PIPE && ok && n_it > 0) ok = tc::mbar_wait(bar(BB_DVDONE), 0, status, 315);
    tc::tc_fence_after();
    if (ok && n_it > 0) {
      const bool live = gj < P.seq_k;
#pragma unroll 1
      for (int which = 0; which < 2; ++which) {
        __nv_bfloat16* out = which ? P.dk : P.dv;
        const float f = live ? (which ? P.scale : 1.f) : 0.f;
#pragma unroll 1
        for (int cc = 0; cc < HD / 64; ++cc) {
          const int c0 = part * (HD / 4) + cc * 16;
          uint32_t o[16];
          tc::tmem_ld16(lane_addr + (which ? DK_COL : DV_COL) + c0, o);   // warp-collective: no lane may skip it
          tc::tmem_ld_wait();
          if (gj < P.t_pad_k) {
            const int col = g * HD + c0;
            __nv_bfloat16* dst = out + ((long long)(col / 64) * P.n_pad_k + row0k + gj) * 64 + (col % 64);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              uint4 v;
              v.x = tc::pack_bf16(__uint_as_float(o[k * 8 + 0]) * f, __uint_as_float(o[k * 8 + 1]) * f);
              v.y = tc::pack_bf16(__uint_as_float(o[k * 8 + 2]) * f, __uint_as_float(o[k * 8 + 3]) * f);
              v.z = tc::pack_bf16(__uint_as_float(o[k * 8 + 4]) * f, __uint_as_float(o[k * 8 + 5]) * f);
              v.w = tc::pack_bf16(__uint_as_float(o[k * 8 + 6]) * f, __uint_as_float(o[k * 8 + 7]) * f);
              *reinterpret_cast<uint4*>(dst + 8 * k) = v;
            }
          }
        }
      }
    }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

template <int HD>
cudaError_t bwd_launch(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* dA,
                       const float* lse, const float* dvec, float* dqacc, void* dK, void* dV, int32_t* status,
                       cudaStream_t st) {
  AttnBwdParams P;
  memset(&P, 0, sizeof(P));
  const int panels = HD / 64;
  if (!fbl_encode_rtile_map(&P.tq, Q, p->n_pad, p->dq / 64, BQ, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tdo, dA, p->n_pad, p->dq / 64, BQ, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tk, K, p->n_pad_kv, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tv, V, p->n_pad_kv, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_f32_panel_map(&P.tdq, dqacc, p->n_pad, p->dq / 64, BQ)) return cudaErrorInvalidValue;
  P.lse = lse; P.dvec = dvec; P.dqacc = dqacc; P.dk = (__nv_bfloat16*)dK; P.dv = (__nv_bfloat16*)dV;
  P.n_pad = p->n_pad; P.seq = p->d.seq; P.t_pad = p->t_pad; P.hq = p->d.n_q_heads; P.group = p->group;
  P.causal = p->d.causal; P.dkv = p->dkv; P.scale = p->scale; P.status = status;
  P.n_pad_k = p->n_pad_kv; P.seq_k = p->seq_kv; P.t_pad_k = p->t_pad_kv;
  auto k = attn_bwd_tc_kernel<HD>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdSmem<HD>::TOTAL);
  if (e != cudaSuccess) return e;
  P.batch = p->d.batch;
  // Q, dO (bf16) and the fp32 dQ accumulator of the query heads of one KV head.  The HD = 128 variant waits for
  // its single-buffered Q / dO tiles on the critical path, so it keeps the blocks that share those tiles close
  // together (small chunks: L2 hits); the pipelined HD = 64 variant hides that latency and prefers balance.
  P.chunk = chunk_for((long long)p->group * p->d.seq * HD * 8, p->d.n_kv_heads * p->d.batch,
                      BwdSmem<HD>::PIPE ? (96ll << 20) : (8ll << 20));
  dim3 grid((unsigned)(((p->t_pad_kv + BKV - 1) / BKV) * p->d.n_kv_heads * p->d.batch));
  return launch_pdl(k, grid, dim3(BWD_THREADS), BwdSmem<HD>::TOTAL, st, P);
}

}  // namespace

bool attn_fwd_tc_supported(const fbl_plan* p) {
  return p->d.dtype == FBL_DTYPE_BF16 && (p->d.head_dim == 64 || p->d.head_dim == 128) && p->n_pad >= 128 &&
         p->n_pad_kv >= 128;
}
bool attn_bwd_tc_supported(const fbl_plan* p) { return attn_fwd_tc_supported(p); }

cudaError_t launch_attn_fwd_tc(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                               int32_t* status, cudaStream_t st) {
  if (p->d.head_dim == 64) return fwd_launch<64>(p, Q, K, V, A, lse, status, st);
  if (p->d.head_dim == 128) return fwd_launch<128>(p, Q, K, V, A, lse, status, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_attn_bwd_tc(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* A,
                               const void* dA, const float* lse, float* dvec, float* dqacc, void* dQ, void* dK,
                               void* dV, bool dvec_ready, int32_t* status, cudaStream_t st) {
  // dQ accumulator := 0, and D = rowsum(dO * O) unless the dA GEMM's epilogue already produced it
  cudaError_t e = launch_attn_bwd_pre(p, A, dA, dvec, dqacc, dvec_ready, st);
  if (e != cudaSuccess) return e;
  if (p->d.head_dim == 64) e = bwd_launch<64>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, status, st);
  else if (p->d.head_dim == 128) e = bwd_launch<128>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, status, st);
  else e = cudaErrorInvalidValue;
  if (e != cudaSuccess) return e;
  return launch_attn_bwd_post(p, dqacc, dQ, st);                      // fp32 accumulator -> storage dtype
}
