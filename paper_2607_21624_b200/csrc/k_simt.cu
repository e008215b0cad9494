// FP32-arithmetic kernels (plain FFMA, no tensor cores) on R-Tile matrices: the projection GEMMs and
// the fused attention forward/backward.  They are the fp32 storage path (single-pass TF32 cannot
// hold a 1e-4 relative bound) and accept bf16 storage too.  Every operand is addressed through the
// R-Tile element map; "transposed" operands are the same tiles read with swapped index roles.
#include "fbl_internal.h"
#include "pdl.cuh"

namespace {

// ------------------------------------------------------------------------------------------
// GEMM: C[m,n] = sum_terms A_t[m,:] . B_t[:,n] (+ bias[n]) (+ residual), 64x64 tile per block.
// ------------------------------------------------------------------------------------------
constexpr int GB = 64, GK = 16;

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  constexpr int TW = tile_w_of<T>::value;
  __shared__ float As[GK][GB + 4];
  __shared__ float Bs[GK][GB + 4];
  const int m0 = blockIdx.y * GB, n0 = blockIdx.x * GB;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {};
  for (int t = 0; t < g.n_terms; ++t) {
    const GemmTerm tm = g.t[t];
    const T* A = (const T*)tm.a;
    const T* B = (const T*)tm.b;
    for (int k0 = 0; k0 < tm.k; k0 += GK) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int e = threadIdx.x + i * 256;
        // A tile: contiguous along k when stored [m][k], along m when stored [k][m]
        int mm, kk;
        if (!tm.a_trans) { kk = e % GK; mm = e / GK; } else { mm = e % GB; kk = e / GB; }
        float v = 0.f;
        if (m0 + mm < g.m && k0 + kk < tm.k)
          v = to_f(tm.a_trans ? A[rt_off<TW>(tm.a_rpad, k0 + kk, m0 + mm)] : A[rt_off<TW>(tm.a_rpad, m0 + mm, k0 + kk)]);
        As[kk][mm] = v;
        int nn, kb;
        if (!tm.b_trans) { nn = e % GB; kb = e / GB; } else { kb = e % GK; nn = e / GK; }
        float w = 0.f;
        if (n0 + nn < g.n && k0 + kb < tm.k)
          w = to_f(tm.b_trans ? B[rt_off<TW>(tm.b_rpad, n0 + nn, k0 + kb)] : B[rt_off<TW>(tm.b_rpad, k0 + kb, n0 + nn)]);
        Bs[kb][nn] = w;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < GK; ++kk) {
        const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      }
      __syncthreads();
    }
  }
  T* C = (T*)g.c;
  const T* R = (const T*)g.residual;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= g.m) continue;
    const bool pad = g.t_pad > 0 && (m % g.t_pad) >= g.seq;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= g.n) continue;
      const int64_t off = rt_off<TW>(g.c_rpad, m, n);
      float v = acc[i][j];
      if (g.bias) v += g.bias[n];
      if (R) v += to_f(R[off]);
      C[off] = from_f<T>(pad ? 0.f : v);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Attention forward: one block per (64-query tile, head, batch); online row softmax over key tiles.
// ------------------------------------------------------------------------------------------
constexpr int BQ = 64, BKV = 64;

template <typename T, int HD>
__global__ void __launch_bounds__(256) attn_fwd_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                            const T* __restrict__ V, T* __restrict__ A,
                                                            float* __restrict__ lse, int64_t n_pad, int seq, int t_pad,
                                                            int64_t n_pad_k, int seq_k, int t_pad_k,
                                                            int hq, int group, int causal, float scale) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int LD = HD + 1;
  constexpr int ND = HD / 16;
  extern __shared__ float sm[];
  float* Qs = sm;                 // [BQ][LD]
  float* Ks = Qs + BQ * LD;       // [BKV][LD]
  float* Vs = Ks + BKV * LD;      // [BKV][LD]
  float* Ss = Vs + BKV * LD;      // [BQ][BKV+1]
  float* s_alpha = Ss + BQ * (BKV + 1);  // [BQ]
  float* s_m = s_alpha + BQ;
  float* s_l = s_m + BQ;
  const int i0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z, gk = h / group;
  const int64_t row0 = (int64_t)b * t_pad, row0k = (int64_t)b * t_pad_k;   // query-side and key-side rows of this sequence
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  for (int e = threadIdx.x; e < BQ * HD; e += 256) {
    const int i = e / HD, d = e % HD;
    Qs[i * LD + d] = (i0 + i < seq) ? to_f(Q[rt_off<TW>(n_pad, row0 + i0 + i, h * HD + d)]) : 0.f;
  }
  if (threadIdx.x < BQ) { s_m[threadIdx.x] = -INFINITY; s_l[threadIdx.x] = 0.f; }
  float o[4][ND] = {};
  const int j_end = causal ? min(seq_k, i0 + BQ) : seq_k;
  for (int j0 = 0; j0 < j_end; j0 += BKV) {
    __syncthreads();
    for (int e = threadIdx.x; e < BKV * HD; e += 256) {
      const int j = e / HD, d = e % HD;
      const bool ok = j0 + j < seq_k;
      const int64_t off = rt_off<TW>(n_pad_k, row0k + j0 + j, gk * HD + d);
      Ks[j * LD + d] = ok ? to_f(K[off]) : 0.f;
      Vs[j * LD + d] = ok ? to_f(V[off]) : 0.f;
    }
    __syncthreads();
    float s[4][4] = {};
    for (int d = 0; d < HD; ++d) {
      float qv[4], kv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { qv[i] = Qs[(ty * 4 + i) * LD + d]; kv[i] = Ks[(tx * 4 + i) * LD + d]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) s[i][j] = fmaf(qv[i], kv[j], s[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gi = i0 + ty * 4 + i, gj = j0 + tx * 4 + j;
        const bool masked = gj >= seq_k || (causal && gj > gi);
        Ss[(ty * 4 + i) * (BKV + 1) + tx * 4 + j] = masked ? -INFINITY : s[i][j] * scale;
      }
    __syncthreads();
    {  // row softmax update: 4 threads per row, 16 columns each
      const int r = threadIdx.x / 4, part = threadIdx.x % 4;
      float* srow = Ss + r * (BKV + 1) + part * 16;
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 16; ++j) mx = fmaxf(mx, srow[j]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_old = s_m[r];
      const float m_new = fmaxf(m_old, mx);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float p = (m_new == -INFINITY) ? 0.f : expf(srow[j] - m_new);
        srow[j] = p;
        sum += p;
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      __syncwarp();
      if (part == 0) {
        const float alpha = (m_new == -INFINITY) ? 1.f : expf(m_old - m_new);
        s_alpha[r] = alpha;
        s_l[r] = s_l[r] * alpha + sum;
        s_m[r] = m_new;
      }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float al = s_alpha[ty * 4 + i];
#pragma unroll
      for (int dd = 0; dd < ND; ++dd) o[i][dd] *= al;
    }
    for (int j = 0; j < BKV; ++j) {
      float pv[4], vv[ND];
#pragma unroll
      for (int i = 0; i < 4; ++i) pv[i] = Ss[(ty * 4 + i) * (BKV + 1) + j];
#pragma unroll
      for (int dd = 0; dd < ND; ++dd) vv[dd] = Vs[j * LD + tx + 16 * dd];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int dd = 0; dd < ND; ++dd) o[i][dd] = fmaf(pv[i], vv[dd], o[i][dd]);
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty * 4 + i, gi = i0 + r;
    if (gi >= t_pad) continue;
    const bool live = gi < seq;
    const float inv = live ? 1.f / s_l[r] : 0.f;
#pragma unroll
    for (int dd = 0; dd < ND; ++dd)
      A[rt_off<TW>(n_pad, row0 + gi, h * HD + tx + 16 * dd)] = from_f<T>(live ? o[i][dd] * inv : 0.f);
    if (tx == 0) lse[((int64_t)b * hq + h) * t_pad + gi] = live ? s_m[r] + logf(s_l[r]) : 0.f;
  }
}

// D_i = sum_d dO[i,d] * O[i,d] per (batch, head, query): one thread per (row, head), 16-byte loads; consecutive
// threads take consecutive rows, i.e. consecutive 128-byte tile rows of the head's column panel.
template <typename T>
__global__ void rowdot_kernel(const T* __restrict__ dA, const T* __restrict__ A, float* __restrict__ dvec,
                              int64_t n_pad, int t_pad, int hq, int hd, int64_t total) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int V = 16 / (int)sizeof(T);
  pdl_launch_dependents();
  pdl_wait();
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int64_t r = i % n_pad;
  const int h = (int)(i / n_pad);
  float s = 0.f;
  for (int d = 0; d < hd; d += V) {
    const int64_t off = rt_off<TW>(n_pad, r, h * hd + d);
    const uint4 ra = *reinterpret_cast<const uint4*>(dA + off), rb = *reinterpret_cast<const uint4*>(A + off);
    const T* ea = reinterpret_cast<const T*>(&ra);
    const T* eb = reinterpret_cast<const T*>(&rb);
#pragma unroll
    for (int k = 0; k < V; ++k) s = fmaf(to_f(ea[k]), to_f(eb[k]), s);
  }
  const int64_t b = r / t_pad, t = r % t_pad;
  dvec[(b * hq + h) * t_pad + t] = s;
}

// ------------------------------------------------------------------------------------------
// Attention backward: one block per (64-key tile, KV head, batch).  dK and dV accumulate in
// registers over the query-tile loop and over the G query heads of the group (the sequence-axis
// and GQA-group reductions); dQ is a key-axis reduction across blocks, added into an fp32 buffer.
// ------------------------------------------------------------------------------------------
template <typename T, int HD>
__global__ void __launch_bounds__(256) attn_bwd_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K,
                                                            const T* __restrict__ V, const T* __restrict__ dA,
                                                            const float* __restrict__ lse,
                                                            const float* __restrict__ dvec, float* __restrict__ dqacc,
                                                            T* __restrict__ dK, T* __restrict__ dV, int64_t n_pad,
                                                            int seq, int t_pad, int64_t n_pad_k, int seq_k, int t_pad_k, int hq, int group, int causal,
                                                            float scale) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int LD = HD + 1;
  constexpr int ND = HD / 16;
  constexpr int LS = BKV + 1;
  extern __shared__ float sm[];
  float* Ks = sm;
  float* Vs = Ks + BKV * LD;
  float* Qs = Vs + BKV * LD;
  float* Os = Qs + BQ * LD;        // dO tile
  float* Ps = Os + BQ * LD;        // [BQ][LS]
  float* Ds = Ps + BQ * LS;        // dS, [BQ][LS]
  float* s_lse = Ds + BQ * LS;
  float* s_d = s_lse + BQ;
  const int j0 = blockIdx.x * BKV, gk = blockIdx.y, b = blockIdx.z;
  const int64_t row0 = (int64_t)b * t_pad, row0k = (int64_t)b * t_pad_k;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  for (int e = threadIdx.x; e < BKV * HD; e += 256) {
    const int j = e / HD, d = e % HD;
    const bool ok = j0 + j < seq_k;
    const int64_t off = rt_off<TW>(n_pad_k, row0k + j0 + j, gk * HD + d);
    Ks[j * LD + d] = ok ? to_f(K[off]) : 0.f;
    Vs[j * LD + d] = ok ? to_f(V[off]) : 0.f;
  }
  float dk[4][ND] = {}, dv[4][ND] = {};
  const int i_begin = causal ? (j0 / BQ) * BQ : 0;
  for (int hh = 0; hh < group; ++hh) {
    const int h = gk * group + hh;
    for (int i0 = i_begin; i0 < seq; i0 += BQ) {
      __syncthreads();
      for (int e = threadIdx.x; e < BQ * HD; e += 256) {
        const int i = e / HD, d = e % HD;
        const bool ok = i0 + i < seq;
        const int64_t off = rt_off<TW>(n_pad, row0 + i0 + i, h * HD + d);
        Qs[i * LD + d] = ok ? to_f(Q[off]) : 0.f;
        Os[i * LD + d] = ok ? to_f(dA[off]) : 0.f;
      }
      if (threadIdx.x < BQ) {
        const int gi = i0 + threadIdx.x;
        const bool ok = gi < seq;
        s_lse[threadIdx.x] = ok ? lse[((int64_t)b * hq + h) * t_pad + gi] : 0.f;
        s_d[threadIdx.x] = ok ? dvec[((int64_t)b * hq + h) * t_pad + gi] : 0.f;
      }
      __syncthreads();
      float s[4][4] = {}, dp[4][4] = {};
      for (int d = 0; d < HD; ++d) {
        float qv[4], ov[4], kv[4], vv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          qv[i] = Qs[(ty * 4 + i) * LD + d];
          ov[i] = Os[(ty * 4 + i) * LD + d];
          kv[i] = Ks[(tx * 4 + i) * LD + d];
          vv[i] = Vs[(tx * 4 + i) * LD + d];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            s[i][j] = fmaf(qv[i], kv[j], s[i][j]);
            dp[i][j] = fmaf(ov[i], vv[j], dp[i][j]);
          }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int li = ty * 4 + i, lj = tx * 4 + j;
          const int gi = i0 + li, gj = j0 + lj;
          const bool masked = gi >= seq || gj >= seq_k || (causal && gj > gi);
          const float p = masked ? 0.f : expf(s[i][j] * scale - s_lse[li]);
          Ps[li * LS + lj] = p;
          Ds[li * LS + lj] = p * (dp[i][j] - s_d[li]);
        }
      __syncthreads();
      // dV[j,d] += sum_i P[i,j] dO[i,d];  dK[j,d] += sum_i dS[i,j] Q[i,d]   (P^T, dS^T by index roles)
      for (int i = 0; i < BQ; ++i) {
        float pv[4], sv[4], ov[ND], qv[ND];
#pragma unroll
        for (int j = 0; j < 4; ++j) { pv[j] = Ps[i * LS + ty * 4 + j]; sv[j] = Ds[i * LS + ty * 4 + j]; }
#pragma unroll
        for (int dd = 0; dd < ND; ++dd) { ov[dd] = Os[i * LD + tx + 16 * dd]; qv[dd] = Qs[i * LD + tx + 16 * dd]; }
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int dd = 0; dd < ND; ++dd) {
            dv[j][dd] = fmaf(pv[j], ov[dd], dv[j][dd]);
            dk[j][dd] = fmaf(sv[j], qv[dd], dk[j][dd]);
          }
      }
      // dQ[i,d] += scale * sum_j dS[i,j] K[j,d]
      float dq[4][ND] = {};
      for (int j = 0; j < BKV; ++j) {
        float sv[4], kv[ND];
#pragma unroll
        for (int i = 0; i < 4; ++i) sv[i] = Ds[(ty * 4 + i) * LS + j];
#pragma unroll
        for (int dd = 0; dd < ND; ++dd) kv[dd] = Ks[j * LD + tx + 16 * dd];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int dd = 0; dd < ND; ++dd) dq[i][dd] = fmaf(sv[i], kv[dd], dq[i][dd]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int gi = i0 + ty * 4 + i;
        if (gi >= seq) continue;
#pragma unroll
        for (int dd = 0; dd < ND; ++dd)
          atomicAdd(&dqacc[rt_off<TW>(n_pad, row0 + gi, h * HD + tx + 16 * dd)], dq[i][dd] * scale);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int gj = j0 + ty * 4 + j;
    if (gj >= t_pad_k) continue;
    const bool live = gj < seq_k;
#pragma unroll
    for (int dd = 0; dd < ND; ++dd) {
      const int64_t off = rt_off<TW>(n_pad_k, row0k + gj, gk * HD + tx + 16 * dd);
      dK[off] = from_f<T>(live ? dk[j][dd] * scale : 0.f);
      dV[off] = from_f<T>(live ? dv[j][dd] : 0.f);
    }
  }
}

template <typename T>
__global__ void convert_f32_kernel(const float* __restrict__ src, T* __restrict__ dst, int64_t n) {
  // n is a multiple of 4 (whole tile rows)
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t i = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) * 4; i < n; i += (int64_t)gridDim.x * blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(src + i);
    dst[i] = from_f<T>(v.x); dst[i + 1] = from_f<T>(v.y); dst[i + 2] = from_f<T>(v.z); dst[i + 3] = from_f<T>(v.w);
  }
}

// Up to four fp32 buffers rounded to bf16 in one launch (blockIdx.y picks the buffer).
__global__ void convert_f32_group_kernel(ConvertGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  const float* __restrict__ src = g.src[blockIdx.y];
  __nv_bfloat16* __restrict__ dst = (__nv_bfloat16*)g.dst[blockIdx.y];
  const int64_t n = g.n[blockIdx.y];
  for (int64_t i = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) * 4; i < n; i += (int64_t)gridDim.x * blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(src + i);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t*>(&lo); o.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst + i) = o;
  }
}

template <typename T, int HD>
cudaError_t attn_fwd_launch(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                            cudaStream_t st) {
  const size_t sh = (size_t)(3 * 64 * (HD + 1) + 64 * 65 + 3 * 64) * sizeof(float);
  auto k = attn_fwd_simt_kernel<T, HD>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
  if (e != cudaSuccess) return e;
  dim3 grid((p->t_pad + BQ - 1) / BQ, p->d.n_q_heads, p->d.batch);
  k<<<grid, 256, sh, st>>>((const T*)Q, (const T*)K, (const T*)V, (T*)A, lse, p->n_pad, p->d.seq, p->t_pad,
                           p->n_pad_kv, p->seq_kv, p->t_pad_kv,
                           p->d.n_q_heads, p->group, p->d.causal, p->scale);
  return cudaGetLastError();
}

template <typename T, int HD>
cudaError_t attn_bwd_launch(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* dA,
                            const float* lse, const float* dvec, float* dqacc, void* dK, void* dV, cudaStream_t st) {
  const size_t sh = (size_t)(4 * 64 * (HD + 1) + 2 * 64 * 65 + 2 * 64) * sizeof(float);
  auto k = attn_bwd_simt_kernel<T, HD>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
  if (e != cudaSuccess) return e;
  dim3 grid((p->t_pad_kv + BKV - 1) / BKV, p->d.n_kv_heads, p->d.batch);
  k<<<grid, 256, sh, st>>>((const T*)Q, (const T*)K, (const T*)V, (const T*)dA, lse, dvec, dqacc, (T*)dK, (T*)dV,
                           p->n_pad, p->d.seq, p->t_pad, p->n_pad_kv, p->seq_kv, p->t_pad_kv, p->d.n_q_heads, p->group,
                           p->d.causal, p->scale);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm_simt(int dtype, const GemmArgs& g, cudaStream_t st) {
  dim3 grid((g.n + GB - 1) / GB, (g.m + GB - 1) / GB);
  if (dtype == FBL_DTYPE_FP32) gemm_simt_kernel<float><<<grid, 256, 0, st>>>(g);
  else gemm_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(g);
  return cudaGetLastError();
}

cudaError_t launch_attn_fwd_simt(const fbl_plan* p, const void* Q, const void* K, const void* V, void* A, float* lse,
                                 cudaStream_t st) {
  const int hd = p->d.head_dim;
  if (p->d.dtype == FBL_DTYPE_FP32) {
    if (hd == 32) return attn_fwd_launch<float, 32>(p, Q, K, V, A, lse, st);
    if (hd == 64) return attn_fwd_launch<float, 64>(p, Q, K, V, A, lse, st);
    if (hd == 128) return attn_fwd_launch<float, 128>(p, Q, K, V, A, lse, st);
  } else {
    if (hd == 64) return attn_fwd_launch<__nv_bfloat16, 64>(p, Q, K, V, A, lse, st);
    if (hd == 128) return attn_fwd_launch<__nv_bfloat16, 128>(p, Q, K, V, A, lse, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_attn_bwd_pre(const fbl_plan* p, const void* A, const void* dA, float* dvec, float* dqacc,
                                bool dvec_ready, cudaStream_t st) {
  const int hd = p->d.head_dim;
  const int64_t total = p->n_pad * p->d.n_q_heads;
  // dqacc was zero-filled with the status word at the start of the step
  (void)dqacc;
  if (dvec_ready) return cudaSuccess;
  const unsigned rb = (unsigned)((total + 255) / 256);
  if (p->d.dtype == FBL_DTYPE_FP32)
    return launch_pdl(rowdot_kernel<float>, dim3(rb), dim3(256), 0, st, (const float*)dA, (const float*)A, dvec, p->n_pad,
                      p->t_pad, p->d.n_q_heads, hd, total);
  return launch_pdl(rowdot_kernel<__nv_bfloat16>, dim3(rb), dim3(256), 0, st, (const __nv_bfloat16*)dA,
                    (const __nv_bfloat16*)A, dvec, p->n_pad, p->t_pad, p->d.n_q_heads, hd, total);
}

cudaError_t launch_attn_bwd_post(const fbl_plan* p, const float* dqacc, void* dQ, cudaStream_t st) {
  const int64_t nq = p->n_pad * p->dq;
  const int blocks = (int)min((int64_t)148 * 8, (nq / 4 + 255) / 256);
  if (p->d.dtype == FBL_DTYPE_FP32)
    return launch_pdl(convert_f32_kernel<float>, dim3(blocks), dim3(256), 0, st, dqacc, (float*)dQ, nq);
  return launch_pdl(convert_f32_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, dqacc, (__nv_bfloat16*)dQ, nq);
}

cudaError_t launch_convert_f32_group(const ConvertGroup& g, cudaStream_t st) {
  int64_t mx = 0;
  for (int i = 0; i < g.count; ++i) mx = g.n[i] > mx ? g.n[i] : mx;
  const int blocks = (int)min((int64_t)148 * 4, (mx / 4 + 255) / 256);
  return launch_pdl(convert_f32_group_kernel, dim3(blocks > 0 ? blocks : 1, g.count), dim3(256), 0, st, g);
}

cudaError_t launch_attn_bwd_simt(const fbl_plan* p, const void* Q, const void* K, const void* V, const void* A,
                                 const void* dA, const float* lse, float* dvec, float* dqacc, void* dQ, void* dK,
                                 void* dV, cudaStream_t st) {
  const int hd = p->d.head_dim;
  cudaError_t e = launch_attn_bwd_pre(p, A, dA, dvec, dqacc, false, st);
  if (e != cudaSuccess) return e;
  e = cudaErrorInvalidValue;
  if (p->d.dtype == FBL_DTYPE_FP32) {
    if (hd == 32) e = attn_bwd_launch<float, 32>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, st);
    else if (hd == 64) e = attn_bwd_launch<float, 64>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, st);
    else if (hd == 128) e = attn_bwd_launch<float, 128>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, st);
  } else {
    if (hd == 64) e = attn_bwd_launch<__nv_bfloat16, 64>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, st);
    else if (hd == 128) e = attn_bwd_launch<__nv_bfloat16, 128>(p, Q, K, V, dA, lse, dvec, dqacc, dK, dV, st);
  }
  if (e != cudaSuccess) return e;
  return launch_attn_bwd_post(p, dqacc, dQ, st);
}
