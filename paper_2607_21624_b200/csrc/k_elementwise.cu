// HBM-bound kernels on R-Tile matrices: pack/unpack, norm forward/backward, token-axis column sums.
// Thread mapping shared by all of them: 8 consecutive lanes cover one 128-byte tile row with one
// 16-byte vector each, 4 rows per warp are 512 contiguous bytes, so every warp-level access is a
// run of whole 128-byte lines.
#include <math.h>

#include "fbl_internal.h"
#include "pdl.cuh"

namespace {

template <typename T> struct Vec16 { static constexpr int N = 16 / (int)sizeof(T); };

template <typename T>
__device__ __forceinline__ void load16(const T* p, float (&v)[Vec16<T>::N]) {
  uint4 raw = *reinterpret_cast<const uint4*>(p);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < Vec16<T>::N; ++i) v[i] = to_f(e[i]);
}
template <typename T>
__device__ __forceinline__ void store16(T* p, const float (&v)[Vec16<T>::N]) {
  uint4 raw;
  T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
  for (int i = 0; i < Vec16<T>::N; ++i) e[i] = from_f<T>(v[i]);
  *reinterpret_cast<uint4*>(p) = raw;
}

__device__ __forceinline__ float group8_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  return v;
}

// ------------------------------------------------------------------------------------------
// pack / unpack: the only layout conversions, used at the graph boundary.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void pack_kernel(const T* __restrict__ src, T* __restrict__ dst, int64_t outer, int64_t rows,
                            int64_t rows_pad, int cols, int64_t total) {
  constexpr int TW = tile_w_of<T>::value;
  const int64_t r_pad = outer * rows_pad;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t panel = i / (r_pad * TW);
    int64_t rem = i - panel * r_pad * TW;
    int64_t r = rem / TW;
    int c = (int)(panel * TW + rem % TW);
    int64_t o = r / rows_pad, row = r - o * rows_pad;
    T v = from_f<T>(0.f);
    if (row < rows) v = src[(o * rows + row) * cols + c];
    dst[i] = v;
  }
}

template <typename T>
__global__ void unpack_kernel(const T* __restrict__ src, T* __restrict__ dst, int64_t outer, int64_t rows,
                              int64_t rows_pad, int cols, int64_t total) {
  constexpr int TW = tile_w_of<T>::value;
  const int64_t r_pad = outer * rows_pad;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t orow = i / cols;
    int c = (int)(i - orow * cols);
    int64_t o = orow / rows, row = orow - o * rows;
    dst[i] = src[rt_off<TW>(r_pad, o * rows_pad + row, c)];
  }
}

// ------------------------------------------------------------------------------------------
// Pre-norm forward: row (feature-axis) reductions.  32 token rows per block.
// stats[2r] = mean (0 for RMSNorm), stats[2r+1] = rstd.  Padding rows get zeros.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) norm_fwd_kernel(const T* __restrict__ X, const float* __restrict__ gamma,
                                                       const float* __restrict__ beta, T* __restrict__ Xn,
                                                       float* __restrict__ stats, int64_t n_pad, int d, int seq,
                                                       int t_pad, int rms, float eps) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int V = Vec16<T>::N;
  const int64_t r = (int64_t)blockIdx.x * 32 + threadIdx.x / 8;
  const int l8 = threadIdx.x % 8;
  if (r >= n_pad) return;                       // whole 8-lane groups leave together
  const bool pad = (int)(r % t_pad) >= seq;
  const int panels = d / TW;
  float v[V];
  float mean = 0.f;
  if (!rms) {
    float s = 0.f;
    for (int p = 0; p < panels; ++p) {
      load16(X + ((int64_t)p * n_pad + r) * TW + l8 * V, v);
#pragma unroll
      for (int i = 0; i < V; ++i) s += v[i];
    }
    mean = group8_sum(s) / (float)d;
  }
  float q = 0.f;
  for (int p = 0; p < panels; ++p) {
    load16(X + ((int64_t)p * n_pad + r) * TW + l8 * V, v);
#pragma unroll
    for (int i = 0; i < V; ++i) { float c = v[i] - mean; q += c * c; }
  }
  float rstd = rsqrtf(group8_sum(q) / (float)d + eps);
  if (pad) { mean = 0.f; rstd = 0.f; }
  if (l8 == 0) { stats[2 * r] = mean; stats[2 * r + 1] = rstd; }
  for (int p = 0; p < panels; ++p) {
    const int64_t off = ((int64_t)p * n_pad + r) * TW + l8 * V;
    load16(X + off, v);
    const int c0 = p * TW + l8 * V;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      float y = (v[i] - mean) * rstd * gamma[c0 + i] + (beta ? beta[c0 + i] : 0.f);
      v[i] = pad ? 0.f : y;
    }
    store16(Xn + off, v);
  }
}

// ------------------------------------------------------------------------------------------
// Pre-norm backward.  Row reductions mean(g), mean(g*xhat) with g = dXn*gamma give dX; the
// token-axis reductions dgamma = sum dXn*xhat and dbeta = sum dXn are accumulated per block in
// shared memory (a reduction over the block's 4 storage tiles) and added to the fp32 outputs.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) norm_bwd_kernel(const T* __restrict__ dXn, const T* __restrict__ X,
                                                       const T* __restrict__ dY, const float* __restrict__ stats,
                                                       const float* __restrict__ gamma, T* __restrict__ dX,
                                                       float* __restrict__ dgamma, float* __restrict__ dbeta,
                                                       int64_t n_pad, int d, int rms) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int V = Vec16<T>::N;
  extern __shared__ float sh[];                 // [2][d]
  float* s_dg = sh;
  float* s_db = sh + d;
  for (int i = threadIdx.x; i < 2 * d; i += blockDim.x) sh[i] = 0.f;
  __syncthreads();
  const int64_t r = (int64_t)blockIdx.x * 32 + threadIdx.x / 8;
  const int l8 = threadIdx.x % 8;
  const bool live = r < n_pad;
  const int panels = d / TW;
  float mean = 0.f, rstd = 0.f;
  if (live) { mean = stats[2 * r]; rstd = stats[2 * r + 1]; }
  float xv[V], gv[V];
  float s1 = 0.f, s2 = 0.f;
  for (int p = 0; p < panels; ++p) {
    const int c0 = p * TW + l8 * V;
    float pg[V], pb[V];
    if (live) {
      const int64_t off = ((int64_t)p * n_pad + r) * TW + l8 * V;
      load16(X + off, xv);
      load16(dXn + off, gv);
#pragma unroll
      for (int i = 0; i < V; ++i) {
        float xh = (xv[i] - mean) * rstd;
        float g = gv[i] * gamma[c0 + i];
        s1 += g;
        s2 += g * xh;
        pg[i] = gv[i] * xh;
        pb[i] = gv[i];
      }
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i) { pg[i] = 0.f; pb[i] = 0.f; }
    }
    // sum the 4 rows of this warp, then one shared-memory add per column per warp
#pragma unroll
    for (int i = 0; i < V; ++i) {
      pg[i] += __shfl_xor_sync(0xffffffffu, pg[i], 8);
      pg[i] += __shfl_xor_sync(0xffffffffu, pg[i], 16);
      pb[i] += __shfl_xor_sync(0xffffffffu, pb[i], 8);
      pb[i] += __shfl_xor_sync(0xffffffffu, pb[i], 16);
    }
    if ((threadIdx.x & 31) < 8) {
#pragma unroll
      for (int i = 0; i < V; ++i) {
        atomicAdd(&s_dg[c0 + i], pg[i]);
        atomicAdd(&s_db[c0 + i], pb[i]);
      }
    }
  }
  s1 = group8_sum(s1) / (float)d;
  s2 = group8_sum(s2) / (float)d;
  if (rms) s1 = 0.f;
  if (live) {
    for (int p = 0; p < panels; ++p) {
      const int64_t off = ((int64_t)p * n_pad + r) * TW + l8 * V;
      const int c0 = p * TW + l8 * V;
      load16(X + off, xv);
      load16(dXn + off, gv);
      float rv[V];
      if (dY) load16(dY + off, rv);
#pragma unroll
      for (int i = 0; i < V; ++i) {
        float xh = (xv[i] - mean) * rstd;
        float o = rstd * (gv[i] * gamma[c0 + i] - s1 - xh * s2);
        xv[i] = dY ? o + rv[i] : o;
      }
      store16(dX + off, xv);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    atomicAdd(&dgamma[i], s_dg[i]);
    if (dbeta) atomicAdd(&dbeta[i], s_db[i]);
  }
}


// ------------------------------------------------------------------------------------------
// Register-resident norm kernels for bf16 rows (NV vectors of 16 bytes per lane, WPR warps per row, d_model =
// 256 NV WPR up to 4096): a warp owns a row or a contiguous part of it, lane l holds vectors l, l + 32, ... of it (each warp-level load covers four
// whole 128-byte tile rows, one per column panel), so X (and dXn) cross HBM exactly once.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// WPR warps share a row (d_model = NV * 256 * WPR columns): the row statistics are combined through shared memory.
// The warps of a row meet at a named barrier of their own (rows of one block do not wait for each other), and
// successive reductions alternate between two exchange buffers: a warp that writes buffer b again has passed the
// barrier of the reduction in between, which every reader of the earlier value reached after reading it.
template <int WPR>
__device__ __forceinline__ float row_sum(float v, float* s_part, int slot, int part, int& buf) {
  v = warp_sum(v);
  if (WPR == 1) return v;
  float* ex = s_part + buf * 8;
  buf ^= 1;
  if ((threadIdx.x & 31) == 0) ex[slot * WPR + part] = v;
  asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "r"(WPR * 32) : "memory");
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < WPR; ++i) t += ex[slot * WPR + i];
  return t;
}

// Two sums in one exchange.
template <int WPR>
__device__ __forceinline__ void row_sum2(float& a, float& b, float* s_part, int slot, int part, int& buf) {
  a = warp_sum(a);
  b = warp_sum(b);
  if (WPR == 1) return;
  float* ex = s_part + buf * 16;
  buf ^= 1;
  if ((threadIdx.x & 31) == 0) { ex[(slot * WPR + part) * 2] = a; ex[(slot * WPR + part) * 2 + 1] = b; }
  asm volatile("bar.sync %0, %1;" ::"r"(1 + slot), "r"(WPR * 32) : "memory");
  a = 0.f; b = 0.f;
#pragma unroll
  for (int i = 0; i < WPR; ++i) { a += ex[(slot * WPR + i) * 2]; b += ex[(slot * WPR + i) * 2 + 1]; }
}

template <int NV, int WPR>
__global__ void __launch_bounds__(256, 2) norm_fwd_rows_kernel(const __nv_bfloat16* __restrict__ X,
                                                            const float* __restrict__ gamma,
                                                            const float* __restrict__ beta,
                                                            __nv_bfloat16* __restrict__ Xn, float* __restrict__ stats,
                                                            int64_t n_pad, int seq, int t_pad, int rms, float eps,
                                                            int32_t* __restrict__ status) {
  constexpr int D = NV * 256 * WPR;
  constexpr int RPB = 8 / WPR;                       // rows per block pass
  __shared__ float s_part[16];
  // First kernel of the forward pass: it resets the pass's status word (later kernels only write it after a
  // bounded wait of about a second has expired), which saves a fill node in front of the pass.
  if (status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0;
  const int lane = threadIdx.x % 32, wib = threadIdx.x / 32;
  const int slot = wib / WPR, part = wib % WPR;
  int buf = 0;
  pdl_launch_dependents();
  // gamma and beta are inputs of the step: in registers before waiting for the previous kernel
  float gm[NV][8], bt[NV][8];
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int c0 = ((part * NV + j) * 32 + lane) * 8;
    const float4 g0 = *reinterpret_cast<const float4*>(gamma + c0), g1 = *reinterpret_cast<const float4*>(gamma + c0 + 4);
    float4 b0 = make_float4(0.f, 0.f, 0.f, 0.f), b1 = b0;
    if (beta) { b0 = *reinterpret_cast<const float4*>(beta + c0); b1 = *reinterpret_cast<const float4*>(beta + c0 + 4); }
    gm[j][0] = g0.x; gm[j][1] = g0.y; gm[j][2] = g0.z; gm[j][3] = g0.w; gm[j][4] = g1.x; gm[j][5] = g1.y; gm[j][6] = g1.z; gm[j][7] = g1.w;
    bt[j][0] = b0.x; bt[j][1] = b0.y; bt[j][2] = b0.z; bt[j][3] = b0.w; bt[j][4] = b1.x; bt[j][5] = b1.y; bt[j][6] = b1.z; bt[j][7] = b1.w;
  }
  pdl_wait();
  // Each block owns a contiguous range of rows and walks it in order: the PF rows in flight are then neighbours,
  // i.e. in every 64-column panel PF adjacent 128-byte pieces (with a grid-stride walk every piece stood alone).
  constexpr int64_t stride = RPB;
  const int64_t per_block = ((n_pad + gridDim.x - 1) / gridDim.x + RPB - 1) / RPB * RPB;
  const int64_t r_end = min(n_pad, ((int64_t)blockIdx.x + 1) * per_block);
  // lane's vectors of a row: vector index v -> panel v / 8, chunk v % 8
  auto vec_off = [&](int j, int64_t r) {
    const int v = (part * NV + j) * 32 + lane;
    return ((int64_t)(v / 8) * n_pad + r) * 64 + (v % 8) * 8;
  };
  // PF rows ahead are in flight per warp (raw vectors in registers): with one row ahead a block waited ~1.4 us
  // per row on the load of the next one; HBM needs about 10 MB in flight across the GPU
  constexpr int PF = NV == 3 ? 3 : 4;
  int64_t r = (int64_t)blockIdx.x * per_block + slot;
  uint4 ring[PF][NV];
#pragma unroll
  for (int k = 0; k < PF; ++k) {
    if (r + k * stride < r_end) {
#pragma unroll
      for (int j = 0; j < NV; ++j) ring[k][j] = *reinterpret_cast<const uint4*>(X + vec_off(j, r + k * stride));
    }
  }
  bool more = r < r_end;
  while (more) {
#pragma unroll
    for (int k = 0; k < PF; ++k) {
      if (r >= r_end) { more = false; break; }
      const bool pad = (int)(r % t_pad) >= seq;
      float x[NV][8];
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&ring[k][j]);
#pragma unroll
        for (int i = 0; i < 8; ++i) { x[j][i] = __bfloat162float(e[i]); s += x[j][i]; }
      }
      if (r + PF * stride < r_end) {
#pragma unroll
        for (int j = 0; j < NV; ++j) ring[k][j] = *reinterpret_cast<const uint4*>(X + vec_off(j, r + PF * stride));
      }
      const float mean = rms ? 0.f : row_sum<WPR>(s, s_part, slot, part, buf) * (1.f / D);
      float q = 0.f;
#pragma unroll
      for (int j = 0; j < NV; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) { const float c = x[j][i] - mean; q += c * c; }
      const float rstd = rsqrtf(row_sum<WPR>(q, s_part, slot, part, buf) * (1.f / D) + eps);
      if (lane == 0 && part == 0) { stats[2 * r] = pad ? 0.f : mean; stats[2 * r + 1] = pad ? 0.f : rstd; }
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        float y[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) y[i] = pad ? 0.f : (x[j][i] - mean) * rstd * gm[j][i] + bt[j][i];
        store16(Xn + vec_off(j, r), y);
      }
      r += stride;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Rotary position embedding, in place, on two R-Tile matrices at once (Q and K forward; dQ and dK backward with the
// opposite angle).  Half-split pairing: inside a head, element i < hd/2 goes with element i + hd/2, and the pair of
// token t turns by t * base^(-2i/hd).  A thread takes 16 bytes of the low half and the matching 16 bytes of the
// high half (the same row of the same or of the neighbouring 128-byte panel).
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) rope_kernel(T* __restrict__ A, int heads_a, T* __restrict__ B, int heads_b,
                                                   int64_t n_pad, int seq, int t_pad, int hd, float neg2_log2_base_over_hd,
                                                   float sign) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int V = Vec16<T>::N;
  pdl_launch_dependents();
  pdl_wait();
  const int half = hd / 2, vec_per_head = half / V;
  const int64_t per_a = n_pad * heads_a * vec_per_head, total = per_a + n_pad * heads_b * vec_per_head;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const bool second = idx >= per_a;
    T* M = second ? B : A;
    const int heads = second ? heads_b : heads_a;
    int64_t rem = second ? idx - per_a : idx;
    // consecutive threads: consecutive vectors of a row's half-head, then rows (whole 128-byte pieces per warp quarter)
    const int v = (int)(rem % vec_per_head);
    rem /= vec_per_head;
    const int64_t r = rem % n_pad;
    const int h = (int)(rem / n_pad);
    const int t = (int)(r % t_pad);
    if (t >= seq) continue;                                     // padding rows hold zeros and stay zero
    const int c_lo = h * hd + v * V, c_hi = c_lo + half;
    T* plo = M + rt_off<TW>(n_pad, r, c_lo);
    T* phi = M + rt_off<TW>(n_pad, r, c_hi);
    float lo[V], hi[V];
    load16(plo, lo);
    load16(phi, hi);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const float inv_freq = exp2f((float)(v * V + i) * neg2_log2_base_over_hd);
      float sn, cs;
      sincosf((float)t * inv_freq, &sn, &cs);
      sn *= sign;
      const float a = lo[i], b = hi[i];
      lo[i] = a * cs - b * sn;
      hi[i] = b * cs + a * sn;
    }
    store16(plo, lo);
    store16(phi, hi);
  }
}

constexpr int COLSUM_SLAB = 256;

struct ColsumGroup {
  const void* m[4];
  float* out[4];
  int cols[4];
  int64_t part_off[4];      // float offset of each matrix's partials inside the scratch area
  int count;
};

// First stage of a token-axis column sum: the block's (64-column panel p, slab of 256 rows) of matrix `which`,
// 32 storage tiles, reduced to one row of partials.  `red` is 32 x (tile width + 1) floats of shared memory.
template <typename T>
__device__ __forceinline__ void colsum_slab(const ColsumGroup& G, int64_t rows, float* __restrict__ part_base, int p,
                                            int slab, int which, float (*red)[tile_w_of<T>::value + 1]) {
  constexpr int TW = tile_w_of<T>::value;
  constexpr int V = Vec16<T>::N;
  const int cols = G.cols[which];
  if (p * TW >= cols) return;
  const T* M = (const T*)G.m[which];
  float* part = part_base + G.part_off[which];
  const int rr = threadIdx.x / 8, l8 = threadIdx.x % 8;
  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  const int64_t r_end = min((int64_t)(slab + 1) * COLSUM_SLAB, rows);
#pragma unroll 8                              // a slab is eight 32-row steps: all their loads in flight together
  for (int64_t r = (int64_t)slab * COLSUM_SLAB + rr; r < r_end; r += 32) {
    float v[V];
    load16(M + ((int64_t)p * rows + r) * TW + l8 * V, v);
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] += v[i];
  }
#pragma unroll
  for (int i = 0; i < V; ++i) red[rr][l8 * V + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < TW) {
    float s = 0.f;
#pragma unroll 8
    for (int k = 0; k < 32; ++k) s += red[k][threadIdx.x];
    part[(int64_t)slab * cols + p * TW + threadIdx.x] = s;
  }
}

// Shared memory of the kernel below: per warp its private token-axis sums (dgamma and dbeta parts of its columns,
// as float4 slots [which][2 NV][32 lanes]: consecutive lanes, consecutive slots, conflict-free), then gamma.
template <int NV, int WPR>
struct NormBwdSmem {
  static constexpr int D = NV * 256 * WPR;
  static constexpr int ACC_F4_PER_WARP = 2 * 2 * NV * 32;
  static constexpr size_t ACC_BYTES = (size_t)8 * ACC_F4_PER_WARP * 16;
  static constexpr size_t BYTES = ACC_BYTES + (size_t)D * 4;
};

// A warp (or WPR warps) owns a row; the row's X and dXn stay in registers as raw bf16 vectors, and the next row's
// are requested before the current row's two reductions, so X and dXn cross HBM exactly once with a row in flight
// per warp at all times.  The token-axis sums (dgamma, dbeta) of a warp's rows accumulate in its private
// shared-memory slots (registers are better spent on the row in flight).
template <int NV, int WPR>
__global__ void __launch_bounds__(256, 2) norm_bwd_rows_kernel(const __nv_bfloat16* __restrict__ dXn,
                                                            const __nv_bfloat16* __restrict__ X,
                                                            const __nv_bfloat16* __restrict__ dY,
                                                            const float* __restrict__ stats,
                                                            const float* __restrict__ gamma,
                                                            __nv_bfloat16* __restrict__ dX, float* __restrict__ partials,
                                                            int64_t n_pad, int rms, int n_norm, ColsumGroup CG,
                                                            float* __restrict__ cs_part, int cs_panels, int cs_slabs) {
  using SMEM = NormBwdSmem<NV, WPR>;
  constexpr int D = SMEM::D;
  constexpr int RPB = 8 / WPR;
  extern __shared__ __align__(16) uint8_t norm_smem[];
  __shared__ float s_part[32];
  // Blocks behind the first n_norm ones do the first stage of the bias gradients' column sums (one launch less):
  // block n_norm + (which * slabs + slab) * panels + p
  if ((int)blockIdx.x >= n_norm) {
    __shared__ float cs_red[32][65];
    pdl_launch_dependents();
    pdl_wait();
    const int idx = (int)blockIdx.x - n_norm;
    colsum_slab<__nv_bfloat16>(CG, n_pad, cs_part, idx % cs_panels, (idx / cs_panels) % cs_slabs, idx / (cs_panels * cs_slabs), cs_red);
    return;
  }
  float4* s_acc = reinterpret_cast<float4*>(norm_smem);
  float* s_gamma = reinterpret_cast<float*>(norm_smem + SMEM::ACC_BYTES);
  const int lane = threadIdx.x % 32, wib = threadIdx.x / 32;
  const int slot = wib / WPR, part = wib % WPR;
  int buf = 0;
  // gamma is an input of the step: into shared memory before waiting for the GEMM in front; the sums start at zero
  for (int i = threadIdx.x; i < D; i += 256) s_gamma[i] = gamma[i];
  for (int i = threadIdx.x; i < 8 * SMEM::ACC_F4_PER_WARP; i += 256) s_acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();
  pdl_launch_dependents();
  float4* my_acc = s_acc + wib * SMEM::ACC_F4_PER_WARP;       // [which][2 j + h][lane]
  auto vec_off = [&](int j, int64_t r) {
    const int v = (part * NV + j) * 32 + lane;
    return ((int64_t)(v / 8) * n_pad + r) * 64 + (v % 8) * 8;
  };
  pdl_wait();
  // each block owns a contiguous range of rows (neighbouring 128-byte pieces in every panel)
  const int64_t per_block = ((n_pad + n_norm - 1) / n_norm + RPB - 1) / RPB * RPB;
  const int64_t r_end = min(n_pad, ((int64_t)blockIdx.x + 1) * per_block);
  int64_t r = (int64_t)blockIdx.x * per_block + slot;
  uint4 xr[NV], gr[NV];
  float2 st = make_float2(0.f, 0.f);
  if (r < r_end) {
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      xr[j] = *reinterpret_cast<const uint4*>(X + vec_off(j, r));
      gr[j] = *reinterpret_cast<const uint4*>(dXn + vec_off(j, r));
    }
    st = *reinterpret_cast<const float2*>(stats + 2 * r);
  }
  while (r < r_end) {
    const int64_t rn = r + RPB;
    uint4 xn[NV], gn[NV], yr[NV];
    float2 stn = make_float2(0.f, 0.f);
    if (rn < r_end) {
#pragma unroll
      for (int j = 0; j < NV; ++j) {
        xn[j] = *reinterpret_cast<const uint4*>(X + vec_off(j, rn));
        gn[j] = *reinterpret_cast<const uint4*>(dXn + vec_off(j, rn));
      }
      stn = *reinterpret_cast<const float2*>(stats + 2 * rn);
    }
    if (dY) {
#pragma unroll
      for (int j = 0; j < NV; ++j) yr[j] = *reinterpret_cast<const uint4*>(dY + vec_off(j, r));
    }
    const float mean = st.x, rstd = st.y;
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const __nv_bfloat16* xe = reinterpret_cast<const __nv_bfloat16*>(&xr[j]);
      const __nv_bfloat16* ge = reinterpret_cast<const __nv_bfloat16*>(&gr[j]);
      const int c0 = ((part * NV + j) * 32 + lane) * 8;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float4 gm = *reinterpret_cast<const float4*>(s_gamma + c0 + 4 * h);
        const float gmv[4] = {gm.x, gm.y, gm.z, gm.w};
        float4 ag = my_acc[(2 * j + h) * 32 + lane], ab = my_acc[(2 * NV + 2 * j + h) * 32 + lane];
        float* agv = reinterpret_cast<float*>(&ag);
        float* abv = reinterpret_cast<float*>(&ab);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float xh = (__bfloat162float(xe[4 * h + i]) - mean) * rstd;
          const float gv = __bfloat162float(ge[4 * h + i]);
          const float g = gv * gmv[i];
          agv[i] = fmaf(gv, xh, agv[i]);
          abv[i] += gv;
          s1 += g;
          s2 = fmaf(g, xh, s2);
        }
        my_acc[(2 * j + h) * 32 + lane] = ag;
        my_acc[(2 * NV + 2 * j + h) * 32 + lane] = ab;
      }
    }
    row_sum2<WPR>(s1, s2, s_part, slot, part, buf);
    s1 = rms ? 0.f : s1 * (1.f / D);
    s2 *= (1.f / D);
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const __nv_bfloat16* xe = reinterpret_cast<const __nv_bfloat16*>(&xr[j]);
      const __nv_bfloat16* ge = reinterpret_cast<const __nv_bfloat16*>(&gr[j]);
      const __nv_bfloat16* ye = reinterpret_cast<const __nv_bfloat16*>(&yr[j]);
      const int c0 = ((part * NV + j) * 32 + lane) * 8;
      float o[8];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float4 gm = *reinterpret_cast<const float4*>(s_gamma + c0 + 4 * h);
        const float gmv[4] = {gm.x, gm.y, gm.z, gm.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float xh = (__bfloat162float(xe[4 * h + i]) - mean) * rstd;
          const float g = __bfloat162float(ge[4 * h + i]) * gmv[i];
          const float dx = rstd * (g - s1 - xh * s2);
          o[4 * h + i] = dY ? __bfloat162float(ye[4 * h + i]) + dx : dx;
        }
      }
      store16(dX + vec_off(j, r), o);
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) { xr[j] = xn[j]; gr[j] = gn[j]; }
    st = stn;
    r = rn;
  }
  __syncthreads();
  // this block's token-axis partial sums: the RPB warps that share a column range are added, and the row goes to
  // row blockIdx.x of partials[blocks][2][D]; a second kernel adds the rows
  float* mine = partials + (int64_t)blockIdx.x * 2 * D;
  const float* accf = reinterpret_cast<const float*>(s_acc);
  for (int c = threadIdx.x; c < D; c += 256) {
    const int v = c / 8, i = c % 8, ln = v % 32, pj = v / 32, pt = pj / NV, j = pj % NV;
    float sg = 0.f, sb = 0.f;
#pragma unroll
    for (int sl = 0; sl < RPB; ++sl) {
      const float* w = accf + (size_t)(sl * WPR + pt) * SMEM::ACC_F4_PER_WARP * 4;
      sg += w[((2 * j + i / 4) * 32 + ln) * 4 + i % 4];
      sb += w[((2 * NV + 2 * j + i / 4) * 32 + ln) * 4 + i % 4];
    }
    mine[c] = sg;
    if (!rms) mine[D + c] = sb;
  }
}


// dgamma[c] (y = 0) or dbeta[c] (y = 1) = sum over the first kernel's blocks of their partial rows.  Blocks with
// y >= ny_norm finish the bias column sums instead (matrix y - ny_norm: the tree over its slab partials), so that
// the step's two small final reductions share one launch.
__global__ void __launch_bounds__(256) norm_bwd_reduce_kernel(const float* __restrict__ part, int blocks, int d,
                                                              float* __restrict__ dgamma, float* __restrict__ dbeta,
                                                              int ny_norm, ColsumGroup G, const float* __restrict__ cpart,
                                                              int n_slabs) {
  __shared__ float red[8][33];
  pdl_launch_dependents();
  pdl_wait();
  if ((int)blockIdx.y >= ny_norm) {
    const int which = blockIdx.y - ny_norm;
    const int cols = G.cols[which];
    const float* cp = cpart + G.part_off[which];
    for (int c = blockIdx.x * 256 + threadIdx.x; c < cols; c += gridDim.x * 256) {
      float s = 0.f;
#pragma unroll 8
      for (int k = 0; k < n_slabs; ++k) s += cp[(int64_t)k * cols + c];
      G.out[which][c] = s;
    }
    return;
  }
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
  const int c = blockIdx.x * 32 + tx;
  float s = 0.f;
  if (c < d) {
    const float* col = part + (int64_t)blockIdx.y * d + c;
    const int64_t stride = 2 * (int64_t)d;
    int b = ty;
    for (; b + 56 < blocks; b += 64) {          // eight independent loads in flight per thread
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = col[(b + 8 * u) * stride];
#pragma unroll
      for (int u = 0; u < 8; ++u) s += v[u];
    }
    for (; b < blocks; b += 8) s += col[b * stride];
  }
  red[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && c < d) {
#pragma unroll
    for (int k = 1; k < 8; ++k) s += red[k][tx];
    (blockIdx.y == 0 ? dgamma : dbeta)[c] = s;
  }
}

template <int NV, int WPR>
void norm_fwd_rows_launch(const fbl_plan* p, const void* X, const float* gamma, const float* beta, void* Xn,
                          float* stats, int rms, int32_t* status, cudaStream_t st) {
  const int blocks = (int)min((int64_t)p->sm_count * 2, p->n_pad / (8 / WPR));
  launch_pdl(norm_fwd_rows_kernel<NV, WPR>, dim3(blocks), dim3(256), 0, st, (const __nv_bfloat16*)X, gamma,
             rms ? (const float*)nullptr : beta, (__nv_bfloat16*)Xn, stats, p->n_pad, p->d.seq, p->t_pad, rms, p->d.eps, status);
}
template <int NV, int WPR>
void norm_bwd_rows_launch(const fbl_plan* p, const void* dXn, const void* X, const void* dY, const float* stats,
                          const float* gamma, void* dX, float* dgamma, float* dbeta, float* part, int rms,
                          const ColsumGroup& cg, const float* cpart, int n_slabs, cudaStream_t st) {
  const int blocks = (int)min((int64_t)p->sm_count * 2, p->n_pad / (8 / WPR));
  int cs_panels = 0;
  for (int i = 0; i < cg.count; ++i) cs_panels = cg.cols[i] / 64 > cs_panels ? cg.cols[i] / 64 : cs_panels;
  const int cs_blocks = cs_panels * n_slabs * cg.count;
  constexpr size_t smem = NormBwdSmem<NV, WPR>::BYTES;
  cudaFuncSetAttribute(norm_bwd_rows_kernel<NV, WPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  launch_pdl(norm_bwd_rows_kernel<NV, WPR>, dim3(blocks + cs_blocks), dim3(256), smem, st, (const __nv_bfloat16*)dXn,
             (const __nv_bfloat16*)X, (const __nv_bfloat16*)dY, stats, gamma, (__nv_bfloat16*)dX, part, p->n_pad, rms,
             blocks, cg, const_cast<float*>(cpart), cs_panels, n_slabs);
  const int ny = rms ? 1 : 2;
  launch_pdl(norm_bwd_reduce_kernel, dim3((p->d.d_model + 31) / 32, ny + cg.count), dim3(256), 0, st, (const float*)part,
             blocks, p->d.d_model, dgamma, dbeta, ny, cg, cpart, n_slabs);
}

// d_model -> (vectors per lane, warps per row) of the register-resident kernels; false if there is none.  At most
// three vectors per lane: the backward keeps five values per column in registers, and two blocks should fit an SM.
bool norm_rows_shape(int d, int* nv, int* wpr) {
  if (d % 256 != 0) return false;
  switch (d / 256) {
    case 1: *nv = 1; *wpr = 1; return true;
    case 2: *nv = 2; *wpr = 1; return true;
    case 3: *nv = 3; *wpr = 1; return true;
    case 4: *nv = 2; *wpr = 2; return true;
    case 6: *nv = 3; *wpr = 2; return true;
    case 8: *nv = 2; *wpr = 4; return true;
    case 12: *nv = 3; *wpr = 4; return true;
    case 16: *nv = 2; *wpr = 8; return true;
    default: return false;
  }
}

#define FBL_NORM_DISPATCH(CALL)                                        \
  do {                                                                 \
    if (wpr == 1) {                                                    \
      if (nv == 1) CALL(1, 1); else if (nv == 2) CALL(2, 1); else CALL(3, 1); \
    } else if (wpr == 2) {                                             \
      if (nv == 2) CALL(2, 2); else CALL(3, 2);                        \
    } else if (wpr == 4) {                                             \
      if (nv == 2) CALL(2, 4); else CALL(3, 4);                        \
    } else {                                                           \
      CALL(2, 8);                                                      \
    }                                                                  \
  } while (0)

// ------------------------------------------------------------------------------------------
// Token-axis column sums, two stages over tiles: (1) one block per (panel, slab of 256 rows)
// reduces its 32 storage tiles to one row of partials, (2) a tree over slabs.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) colsum_stage1(ColsumGroup G, int64_t rows, float* __restrict__ part_base) {
  __shared__ float red[32][tile_w_of<T>::value + 1];
  pdl_launch_dependents();
  pdl_wait();
  colsum_slab<T>(G, rows, part_base, blockIdx.x, blockIdx.y, blockIdx.z, red);
}

__global__ void colsum_stage2(ColsumGroup G, const float* __restrict__ part_base, int n_slabs) {
  pdl_launch_dependents();
  pdl_wait();
  const int which = blockIdx.y;
  const int cols = G.cols[which];
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  const float* part = part_base + G.part_off[which];
  float s = 0.f;
#pragma unroll 8
  for (int k = 0; k < n_slabs; ++k) s += part[(int64_t)k * cols + c];
  G.out[which][c] = s;
}

}  // namespace

cudaError_t launch_pack(int dtype, int unpack, const void* src, void* dst, int64_t outer, int64_t rows,
                        int64_t rows_pad, int cols, cudaStream_t st) {
  const int64_t total = unpack ? outer * rows * cols : outer * rows_pad * cols;
  if (total == 0) return cudaSuccess;
  const int blocks = (int)min((int64_t)148 * 16, (total + 255) / 256);
  if (dtype == FBL_DTYPE_FP32) {
    if (unpack) unpack_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, (float*)dst, outer, rows, rows_pad, cols, total);
    else pack_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, (float*)dst, outer, rows, rows_pad, cols, total);
  } else {
    using B = __nv_bfloat16;
    if (unpack) unpack_kernel<B><<<blocks, 256, 0, st>>>((const B*)src, (B*)dst, outer, rows, rows_pad, cols, total);
    else pack_kernel<B><<<blocks, 256, 0, st>>>((const B*)src, (B*)dst, outer, rows, rows_pad, cols, total);
  }
  return cudaGetLastError();
}

cudaError_t launch_rope(const fbl_plan* p, void* A, int heads_a, void* B, int heads_b, int inverse, cudaStream_t st) {
  const int hd = p->d.head_dim;
  const float k = -2.f * log2f(p->rope_base) / (float)hd;
  const int vec = p->d.dtype == FBL_DTYPE_FP32 ? 4 : 8;
  const int64_t total = p->n_pad * (int64_t)(heads_a + heads_b) * (hd / 2 / vec);
  const int blocks = (int)min((int64_t)p->sm_count * 16, (total + 255) / 256);
  if (p->d.dtype == FBL_DTYPE_FP32)
    return launch_pdl(rope_kernel<float>, dim3(blocks), dim3(256), 0, st, (float*)A, heads_a, (float*)B, heads_b, p->n_pad,
                      p->d.seq, p->t_pad, hd, k, inverse ? -1.f : 1.f);
  return launch_pdl(rope_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, (__nv_bfloat16*)A, heads_a,
                    (__nv_bfloat16*)B, heads_b, p->n_pad, p->d.seq, p->t_pad, hd, k, inverse ? -1.f : 1.f);
}

bool norm_fwd_resets_status(const fbl_plan* p) {
  int nv, wpr;
  return p->d.dtype == FBL_DTYPE_BF16 && norm_rows_shape(p->d.d_model, &nv, &wpr);
}

cudaError_t launch_norm_fwd(const fbl_plan* p, const void* X, const float* gamma, const float* beta, void* Xn,
                            float* stats, int32_t* status, cudaStream_t st) {
  const int blocks = (int)((p->n_pad + 31) / 32);
  const int rms = p->d.norm == FBL_NORM_RMSNORM;
  int nv, wpr;
  if (p->d.dtype == FBL_DTYPE_BF16 && norm_rows_shape(p->d.d_model, &nv, &wpr)) {
#define FBL_CALL(NV_, WPR_) norm_fwd_rows_launch<NV_, WPR_>(p, X, gamma, beta, Xn, stats, rms, status, st)
    FBL_NORM_DISPATCH(FBL_CALL);
#undef FBL_CALL
    return cudaGetLastError();
  }
  if (p->d.dtype == FBL_DTYPE_FP32)
    norm_fwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)X, gamma, rms ? nullptr : beta, (float*)Xn, stats,
                                                   p->n_pad, p->d.d_model, p->d.seq, p->t_pad, rms, p->d.eps);
  else
    norm_fwd_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)X, gamma, rms ? nullptr : beta,
                                                           (__nv_bfloat16*)Xn, stats, p->n_pad, p->d.d_model,
                                                           p->d.seq, p->t_pad, rms, p->d.eps);
  return cudaGetLastError();
}

// Norm backward, and with it (bias_count > 0, register-resident bf16 path only) the bias column sums of up to four
// matrices: their first stage runs as extra blocks of the norm's rows kernel, their second stage inside the norm's
// own second kernel.
// `part` holds the column-sum slab partials first and the norm's per-block partial rows behind them.
bool norm_bwd_takes_colsums(const fbl_plan* p) {
  int nv, wpr;
  return p->d.dtype == FBL_DTYPE_BF16 && norm_rows_shape(p->d.d_model, &nv, &wpr);
}

cudaError_t launch_norm_bwd(const fbl_plan* p, const void* dXn, const void* X, const void* dY, const float* stats,
                            const float* gamma, void* dX, float* dgamma, float* dbeta, float* part,
                            cudaStream_t st, int bias_count, const void* const* bias_m, const int* bias_cols,
                            float* const* bias_out) {
  const int blocks = (int)((p->n_pad + 31) / 32);
  const int d = p->d.d_model;
  const int rms = p->d.norm == FBL_NORM_RMSNORM;
  const size_t sh = 2 * (size_t)d * sizeof(float);
  int nv, wpr;
  if (p->d.dtype == FBL_DTYPE_BF16 && norm_rows_shape(d, &nv, &wpr)) {
    ColsumGroup cg;
    memset(&cg, 0, sizeof(cg));
    const int n_slabs = (int)((p->n_pad + COLSUM_SLAB - 1) / COLSUM_SLAB);
    float* npart = part;
    if (bias_count > 0) {
      if (bias_count > 4) return cudaErrorInvalidValue;
      int max_cols = 0;
      int64_t off = 0;
      for (int i = 0; i < bias_count; ++i) {
        cg.m[i] = bias_m[i]; cg.out[i] = bias_out[i]; cg.cols[i] = bias_cols[i]; cg.part_off[i] = off;
        off += (int64_t)n_slabs * bias_cols[i];
        max_cols = bias_cols[i] > max_cols ? bias_cols[i] : max_cols;
      }
      cg.count = bias_count;                // their first stage rides in the rows kernel's launch, as extra blocks
      (void)max_cols;
      npart = part + (off + 255) / 256 * 256;
    }
    // token-axis sums in two steps over `npart` (no atomics: the result does not depend on block order)
#define FBL_CALL(NV_, WPR_) norm_bwd_rows_launch<NV_, WPR_>(p, dXn, X, dY, stats, gamma, dX, dgamma, dbeta, npart, rms, cg, part, n_slabs, st)
    FBL_NORM_DISPATCH(FBL_CALL);
#undef FBL_CALL
    return cudaGetLastError();
  }
  if (bias_count > 0) return cudaErrorInvalidValue;      // callers ask norm_bwd_takes_colsums first
  cudaError_t e = cudaMemsetAsync(dgamma, 0, d * sizeof(float), st);
  if (e != cudaSuccess) return e;
  if (dbeta) {
    e = cudaMemsetAsync(dbeta, 0, d * sizeof(float), st);
    if (e != cudaSuccess) return e;
  }
  if (p->d.dtype == FBL_DTYPE_FP32) {
    auto k = norm_bwd_kernel<float>;
    if (sh > 48 * 1024) cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
    k<<<blocks, 256, sh, st>>>((const float*)dXn, (const float*)X, (const float*)dY, stats, gamma, (float*)dX, dgamma,
                               rms ? nullptr : dbeta, p->n_pad, d, rms);
  } else {
    using B = __nv_bfloat16;
    auto k = norm_bwd_kernel<B>;
    if (sh > 48 * 1024) cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
    k<<<blocks, 256, sh, st>>>((const B*)dXn, (const B*)X, (const B*)dY, stats, gamma, (B*)dX, dgamma,
                               rms ? nullptr : dbeta, p->n_pad, d, rms);
  }
  return cudaGetLastError();
}

size_t colsum_scratch_bytes(int64_t rows, int64_t cols) {
  const int64_t slabs = (rows + COLSUM_SLAB - 1) / COLSUM_SLAB;
  return (size_t)(slabs * cols) * sizeof(float);
}

// Column sums of up to four matrices that share a row count, in one pair of launches.
cudaError_t launch_colsum_group(int dtype, int count, const void* const* M, int64_t rows, const int* cols, float* const* out,
                                float* partials, cudaStream_t st) {
  if (count < 1 || count > 4) return cudaErrorInvalidValue;
  const int slabs = (int)((rows + COLSUM_SLAB - 1) / COLSUM_SLAB);
  ColsumGroup G;
  int max_cols = 0;
  int64_t off = 0;
  for (int i = 0; i < count; ++i) {
    G.m[i] = M[i]; G.out[i] = out[i]; G.cols[i] = cols[i]; G.part_off[i] = off;
    off += (int64_t)slabs * cols[i];
    max_cols = cols[i] > max_cols ? cols[i] : max_cols;
  }
  G.count = count;
  const int tw = dtype == FBL_DTYPE_FP32 ? 32 : 64;
  dim3 grid((unsigned)(max_cols / tw), slabs, count);
  cudaError_t e;
  if (dtype == FBL_DTYPE_FP32) e = launch_pdl(colsum_stage1<float>, grid, dim3(256), 0, st, G, rows, partials);
  else e = launch_pdl(colsum_stage1<__nv_bfloat16>, grid, dim3(256), 0, st, G, rows, partials);
  if (e != cudaSuccess) return e;
  dim3 grid2((unsigned)((max_cols + 127) / 128), count);
  return launch_pdl(colsum_stage2, grid2, dim3(128), 0, st, G, (const float*)partials, slabs);
}

cudaError_t launch_colsum(int dtype, const void* M, int64_t rows, int64_t cols, float* out, float* partials,
                          cudaStream_t st) {
  const int c = (int)cols;
  return launch_colsum_group(dtype, 1, &M, rows, &c, &out, partials, st);
}

// ------------------------------------------------------------------------------------------
// Column sums without caller scratch.  The per-slab partial sums live in a fixed array inside the
// library image instead of a caller buffer, for callers that are not in a position to allocate.
// ------------------------------------------------------------------------------------------
#include <mutex>

#define FBL_COLSUM_NOALLOC_MAX_FLOATS (256 * 1024)   // 1 MiB: e.g. 16384 rows x 4096 columns

static __device__ __align__(256) float g_colsum_partials[FBL_COLSUM_NOALLOC_MAX_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
float* g_partials_addr[kMaxDevices] = {};   // device address of g_colsum_partials, per device ordinal
}  // namespace

extern "C" int fbl_colsum_noalloc(const fbl_plan* plan, const void* M_dev, int64_t rows, int64_t cols,
                                  float* out_dev, void* stream) {
  if (!plan || !M_dev || !out_dev || rows <= 0 || cols <= 0 || rows % 8 != 0 || cols % plan->tw != 0)
    return FBL_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(M_dev) & (FBL_ALIGN - 1)) != 0) return FBL_ERR_MISALIGNED;
  const int64_t slabs = (rows + COLSUM_SLAB - 1) / COLSUM_SLAB;
  if (slabs * cols > FBL_COLSUM_NOALLOC_MAX_FLOATS) {
    fbl_note_cuda_error(cudaSuccess, "fbl_colsum_noalloc: ceil(rows/256) * cols exceeds the built-in 262144-float area");
    return FBL_ERR_WORKSPACE_TOO_SMALL;
  }
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    fbl_note_cuda_error(e, "fbl_colsum_noalloc: cudaGetDevice");
    return FBL_ERR_CUDA;
  }
  float* partials = nullptr;
  {
    // Set-up, once per device and with that device current: in host code the array's name is only a
    // handle, so ask the runtime for the address the kernels must be given.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_partials_addr[dev]) {
      void* addr = nullptr;
      e = cudaGetSymbolAddress(&addr, g_colsum_partials);
      if (e != cudaSuccess || !addr) {
        fbl_note_cuda_error(e, "fbl_colsum_noalloc: cudaGetSymbolAddress");
        return FBL_ERR_CUDA;
      }
      g_partials_addr[dev] = static_cast<float*>(addr);
    }
    partials = g_partials_addr[dev];
  }
  // Stage 1 writes every partial that stage 2 reads, so nothing left over from an earlier call is used.
  e = launch_colsum(plan->d.dtype, M_dev, rows, cols, out_dev, partials, reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    fbl_note_cuda_error(e, "fbl_colsum_noalloc: launch");
    return FBL_ERR_CUDA;
  }
  return FBL_OK;
}
