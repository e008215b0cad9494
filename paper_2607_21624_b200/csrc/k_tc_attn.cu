// Fused attention on tcgen05 tensor cores, operands in R-Tile order fetched by TMA.
//
// Forward: one block per (128-query tile, head, batch).  S = Q K^T goes to TMEM (two buffers, so the
// tensor pipe computes the next score tile while the softmax warps work on the current one); the
// softmax warps own one query row per thread, keep the running max / sum, and hand P (bf16) to the
// tensor pipe through 128-byte-swizzled shared memory; O accumulates in TMEM and is rescaled in place
// only when a row's running max moved.  K/V tiles of the group's KV head are addressed by the head map
// g = h / G; the head split of Q, K, V and the merge of O are column-panel coordinates of the TMA
// boxes and of the output rows, no data is rearranged.
#include <string.h>

#include "fbl_internal.h"
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
  float scale;
  int32_t* status;
};

template <int HD>
struct FwdSmem {
  static constexpr uint32_t PANELS = HD / 64;
  static constexpr uint32_t TILE = PANELS * 16384;          // 128 rows x HD bf16
  static constexpr uint32_t Q_OFF = 0;
  static constexpr uint32_t K_OFF = TILE;                   // 2 stages
  static constexpr uint32_t V_OFF = 3 * TILE;               // 2 stages
  static constexpr uint32_t P_OFF = 5 * TILE;               // 128 x 128 bf16
  static constexpr uint32_t BAR_OFF = P_OFF + 32768;
  static constexpr uint32_t N_BARS = 16;
  static constexpr uint32_t TOTAL = BAR_OFF + 8 * N_BARS + 16 + 1024;
};

enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_PFULL = 11, B_PVDONE = 12 };

template <int HD>
__global__ void __launch_bounds__(192, 1) attn_fwd_tc_kernel(const __grid_constant__ AttnFwdParams P) {
  using SM = FwdSmem<HD>;
  constexpr uint32_t PANELS = SM::PANELS;
  constexpr uint32_t S_COL = 0, O_COL = 256, TMEM_COLS = 512;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + SM::BAR_OFF;
  const uint32_t slot = bars + 8 * SM::N_BARS;
  auto bar = [&](int i) { return bars + 8u * i; };
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int n_qt = (P.seq + BQ - 1) / BQ;
  const int qt = n_qt - 1 - (int)blockIdx.x;                 // heaviest (latest) causal tiles first
  const int i0 = qt * BQ, h = blockIdx.y, b = blockIdx.z, g = h / P.group;
  const int row0 = b * P.t_pad;
  const int kv_end = P.causal ? min(P.seq, i0 + BQ) : P.seq;
  const int n_kv = (kv_end + BKV - 1) / BKV;
  int32_t* status = P.status;

  if (threadIdx.x == 0) {
    tc::mbar_init(bar(B_QFULL), 1);
    for (int s = 0; s < 2; ++s) {
      tc::mbar_init(bar(B_KFULL + s), 1);
      tc::mbar_init(bar(B_KEMPTY + s), 1);
      tc::mbar_init(bar(B_VFULL + s), 1);
      tc::mbar_init(bar(B_VEMPTY + s), 1);
      tc::mbar_init(bar(B_SFULL + s), 1);
    }
    tc::mbar_init(bar(B_PFULL), 128);
    tc::mbar_init(bar(B_PVDONE), 1);
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

  if (warp == 0 && lane == 0) {
    // ---- TMA producer ------------------------------------------------------------------------
    tc::tma_prefetch_desc(&P.tq);
    tc::tma_prefetch_desc(&P.tk);
    tc::tma_prefetch_desc(&P.tv);
    tc::mbar_expect_tx(bar(B_QFULL), SM::TILE);
    tc::tma_load_3d(base + SM::Q_OFF, &P.tq, bar(B_QFULL), 0, row0 + i0, h * (int)PANELS);
    for (int j = 0; j < n_kv; ++j) {
      const int s = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      if (!tc::mbar_wait(bar(B_KEMPTY + s), ph ^ 1, status, 201)) break;
      tc::mbar_expect_tx(bar(B_KFULL + s), SM::TILE);
      tc::tma_load_3d(base + SM::K_OFF + s * SM::TILE, &P.tk, bar(B_KFULL + s), 0, row0 + j * BKV, g * (int)PANELS);
      if (!tc::mbar_wait(bar(B_VEMPTY + s), ph ^ 1, status, 202)) break;
      tc::mbar_expect_tx(bar(B_VFULL + s), SM::TILE);
      tc::tma_load_3d(base + SM::V_OFF + s * SM::TILE, &P.tv, bar(B_VFULL + s), 0, row0 + j * BKV, g * (int)PANELS);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer --------------------------------------------------------------------------
    const uint32_t idesc_s = tc::idesc_bf16(BQ, BKV, 0, 0);          // Q K-major, K K-major
    const uint32_t idesc_o = tc::idesc_bf16(BQ, HD, 0, 1);           // P K-major, V MN-major (rows are keys)
    auto issue_s = [&](int j) {
      const uint32_t ksm = base + SM::K_OFF + (j & 1) * SM::TILE;
#pragma unroll
      for (uint32_t kk = 0; kk < HD / 16; ++kk) {
        const uint32_t o = (kk / 4) * 16384 + (kk % 4) * 32;
        tc::mma_bf16_ss(tmem_base + S_COL + (j & 1) * 128, tc::smem_desc_sw128(base + SM::Q_OFF + o, 16, 1024),
                        tc::smem_desc_sw128(ksm + o, 16, 1024), idesc_s, kk > 0);
      }
      tc::mma_commit(bar(B_SFULL + (j & 1)));
      tc::mma_commit(bar(B_KEMPTY + (j & 1)));
    };
    bool ok = tc::mbar_wait(bar(B_QFULL), 0, status, 203) && tc::mbar_wait(bar(B_KFULL), 0, status, 204);
    if (ok) {
      tc::tc_fence_after();
      issue_s(0);
    }
    for (int j = 0; j < n_kv && ok; ++j) {
      if (j + 1 < n_kv) {
        if (!tc::mbar_wait(bar(B_KFULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, status, 205)) { ok = false; break; }
        tc::tc_fence_after();
        issue_s(j + 1);
      }
      if (!tc::mbar_wait(bar(B_PFULL), j & 1, status, 206)) { ok = false; break; }
      if (!tc::mbar_wait(bar(B_VFULL + (j & 1)), (j >> 1) & 1, status, 207)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t vsm = base + SM::V_OFF + (j & 1) * SM::TILE;
#pragma unroll
      for (uint32_t kk = 0; kk < BKV / 16; ++kk) {
        const uint64_t da = tc::smem_desc_sw128(base + SM::P_OFF + (kk / 4) * 16384 + (kk % 4) * 32, 16, 1024);
        const uint64_t db = tc::smem_desc_sw128(vsm + kk * 2048, 16384, 1024);
        tc::mma_bf16_ss(tmem_base + O_COL, da, db, idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
      }
      tc::mma_commit(bar(B_PVDONE));
      tc::mma_commit(bar(B_VEMPTY + (j & 1)));
    }
  } else if (warp >= 2) {
    // ---- softmax warps: one query row per thread ----------------------------------------------
    const int q = warp % 4;
    const int r = q * 32 + lane;
    const int gi = i0 + r;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const float c = P.scale * LOG2E;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv && ok; ++j) {
      const int j0 = j * BKV;
      if (!tc::mbar_wait(bar(B_SFULL + (j & 1)), (j >> 1) & 1, status, 208)) { ok = false; break; }
      tc::tc_fence_after();
      uint32_t sr[128];
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) tc::tmem_ld32(lane_addr + S_COL + (j & 1) * 128 + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[cc * 32]));
      tc::tmem_ld_wait();
      float* s = reinterpret_cast<float*>(sr);
      const bool need_mask = (j0 + BKV > P.seq) || (P.causal && j0 + BKV - 1 > i0);
      if (need_mask) {
#pragma unroll
        for (int k = 0; k < 128; ++k) {
          const int gj = j0 + k;
          if (gj >= P.seq || (P.causal && gj > gi)) s[k] = -INFINITY;
        }
      }
      float mx = s[0];
#pragma unroll
      for (int k = 1; k < 128; ++k) mx = fmaxf(mx, s[k]);
      const float m_new = fmaxf(m, mx);
      const bool moved = m_new > m;
      const float alpha = (m == -INFINITY) ? 0.f : tc::fast_exp2((m - m_new) * c);
      const float mc = (m_new == -INFINITY) ? 0.f : m_new * c;
      float sum = 0.f;
#pragma unroll
      for (int k = 0; k < 128; ++k) {
        s[k] = tc::fast_exp2(fmaf(s[k], c, -mc));
        sum += s[k];
      }
      l = l * alpha + sum;
      m = m_new;
      if (j > 0) {
        // the previous P V product must have finished before P is overwritten or O is touched
        if (!tc::mbar_wait(bar(B_PVDONE), (j - 1) & 1, status, 209)) { ok = false; break; }
        tc::tc_fence_after();
        if (__any_sync(0xffffffffu, moved)) {
          const float a = moved ? alpha : 1.f;
#pragma unroll
          for (int cc = 0; cc < HD / 32; ++cc) {
            uint32_t o[32];
            tc::tmem_ld32(lane_addr + O_COL + cc * 32, o);
            tc::tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * a);
            tc::tmem_st32(lane_addr + O_COL + cc * 32, o);
          }
          tc::tmem_st_wait();
        }
      }
      // P row -> shared memory in the 128-byte-swizzled K-major operand layout (two 64-key panels)
#pragma unroll
      for (int ch = 0; ch < 16; ++ch) {
        uint4 v;
        v.x = tc::pack_bf16(s[ch * 8 + 0], s[ch * 8 + 1]);
        v.y = tc::pack_bf16(s[ch * 8 + 2], s[ch * 8 + 3]);
        v.z = tc::pack_bf16(s[ch * 8 + 4], s[ch * 8 + 5]);
        v.w = tc::pack_bf16(s[ch * 8 + 6], s[ch * 8 + 7]);
        const uint32_t addr = base + SM::P_OFF + (ch / 8) * 16384 + r * 128 + (((ch % 8) ^ (r & 7)) * 16);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
      }
      tc::fence_proxy_async();
      tc::tc_fence_before();
      tc::mbar_arrive(bar(B_PFULL));
    }
    if (ok && n_kv > 0) ok = tc::mbar_wait(bar(B_PVDONE), (n_kv - 1) & 1, status, 210);
    tc::tc_fence_after();
    if (ok) {
      const bool live = gi < P.seq;
      const float inv = live ? 1.f / l : 0.f;
#pragma unroll
      for (int cc = 0; cc < HD / 32; ++cc) {
        uint32_t o[32];
        tc::tmem_ld32(lane_addr + O_COL + cc * 32, o);
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

template <int HD>
cudaError_t fwd_launch(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                       int32_t* status, cudaStream_t st) {
  AttnFwdParams P;
  memset(&P, 0, sizeof(P));
  const int panels = HD / 64;
  if (!fbl_encode_rtile_map(&P.tq, Q, p->n_pad, p->dq / 64, BQ, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tk, K, p->n_pad, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  if (!fbl_encode_rtile_map(&P.tv, V, p->n_pad, p->dkv / 64, BKV, panels)) return cudaErrorInvalidValue;
  P.a = (__nv_bfloat16*)A; P.lse = lse; P.n_pad = p->n_pad;
  P.seq = p->d.seq; P.t_pad = p->t_pad; P.hq = p->d.n_q_heads; P.group = p->group; P.causal = p->d.causal;
  P.scale = p->scale; P.status = status;
  auto k = attn_fwd_tc_kernel<HD>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FwdSmem<HD>::TOTAL);
  if (e != cudaSuccess) return e;
  dim3 grid((p->d.seq + BQ - 1) / BQ, p->d.n_q_heads, p->d.batch);
  k<<<grid, 192, FwdSmem<HD>::TOTAL, st>>>(P);
  return cudaGetLastError();
}

}  // namespace

bool attn_fwd_tc_supported(const fbl_plan* p) {
  return p->d.dtype == FBL_DTYPE_BF16 && (p->d.head_dim == 64 || p->d.head_dim == 128) && p->n_pad >= 128;
}
bool attn_bwd_tc_supported(const fbl_plan*) { return false; }

cudaError_t launch_attn_fwd_tc(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                               int32_t* status, cudaStream_t st) {
  if (p->d.head_dim == 64) return fwd_launch<64>(p, Q, K, V, A, lse, status, st);
  if (p->d.head_dim == 128) return fwd_launch<128>(p, Q, K, V, A, lse, status, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_attn_bwd_tc(const fbl_plan*, const void*, const void*, const void*, const void*, const void*,
                               const float*, float*, float*, void*, void*, void*, int32_t*, cudaStream_t) {
  return cudaErrorNotSupported;
}
