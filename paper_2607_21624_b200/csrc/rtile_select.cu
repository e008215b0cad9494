// Offline storage-tile candidate generation: the paper's progressive filter (computation, memory, tensor shape)
// with this GPU's constants in place of the texture-cache ones.  Host code only.
#include <algorithm>
#include <vector>

#include "fbl_internal.h"

namespace {

constexpr int LINE_BYTES = 128;        // L2 line = one row of the 128-byte swizzle atom = the cache tile of Eq. 1 (C_h = 1)
constexpr int SWIZZLE_ROWS = 8;        // rows of the swizzle atom
constexpr int COMPUTE_TILE_ROWS = 128; // rows of an MMA operand tile
constexpr int MAX_TILE_BYTES = 4096;

struct Cand { int h, w, n_cache; double pad; };

double pad_ratio_of(int h, int w, const int64_t* shapes, int n) {
  double worst = 0.0;
  for (int i = 0; i < n; ++i) {
    const int64_t r = shapes[2 * i], c = shapes[2 * i + 1];
    const int64_t rp = (r + h - 1) / h * h, cp = (c + w - 1) / w * w;
    const double ratio = (double)(rp * cp) / (double)(r * c) - 1.0;
    worst = std::max(worst, ratio);
  }
  return worst;
}

}  // namespace

extern "C" int fbl_rtile_candidates(const int64_t* shapes, int n_shapes, int elem_bytes, float max_pad_ratio,
                                    fbl_rtile_cand* out, int max_out, int32_t reject_counts[3]) {
  if (!shapes || n_shapes <= 0 || !out || max_out <= 0 || (elem_bytes != 2 && elem_bytes != 4) || !(max_pad_ratio >= 0.f))
    return FBL_ERR_INVALID_ARG;
  for (int i = 0; i < 2 * n_shapes; ++i) if (shapes[i] <= 0) return FBL_ERR_INVALID_ARG;
  static const int hs[] = {1, 2, 4, 8, 16, 32, 64, 128};
  static const int wbytes[] = {32, 64, 128, 256, 512};
  int rej[3] = {0, 0, 0};
  std::vector<Cand> keep;
  for (int h : hs)
    for (int wb : wbytes) {
      const int w = wb / elem_bytes;
      // C1 (computation): descriptor-compatible row span, whole swizzle atoms, divides the compute tile
      const bool c1 = wb == LINE_BYTES && h % SWIZZLE_ROWS == 0 && COMPUTE_TILE_ROWS % h == 0;
      if (!c1) { ++rej[0]; continue; }
      // C2 (memory): whole lines, bounded tile
      const bool c2 = wb % LINE_BYTES == 0 && h * wb <= MAX_TILE_BYTES;
      if (!c2) { ++rej[1]; continue; }
      // C3 (shape): padding
      const double pad = pad_ratio_of(h, w, shapes, n_shapes);
      if (pad > (double)max_pad_ratio) { ++rej[2]; continue; }
      keep.push_back({h, w, h * ((wb + LINE_BYTES - 1) / LINE_BYTES), pad});     // Eq. 1 with C_h = 1, C_w = one line
    }
  std::sort(keep.begin(), keep.end(), [](const Cand& a, const Cand& b) {
    return a.n_cache != b.n_cache ? a.n_cache < b.n_cache : a.pad < b.pad;
  });
  const int n = (int)std::min<size_t>(keep.size(), (size_t)max_out);
  for (int i = 0; i < n; ++i) out[i] = {keep[i].h, keep[i].w, keep[i].n_cache, (float)keep[i].pad};
  if (reject_counts) { reject_counts[0] = rej[0]; reject_counts[1] = rej[1]; reject_counts[2] = rej[2]; }
  return (int)keep.size();
}
