// Block numbering shared by the attention kernels.
#pragma once

// (head, batch) pairs are taken in chunks small enough for their operands to stay in L2 together; inside a chunk the
// causal-work index ("slot": query-tile slot forward, key tile backward) varies slowest, heaviest first, so the
// block scheduler, which dispatches in block-id order, hands out the long blocks of a chunk before its short ones.
__device__ __forceinline__ void decode_block(int lin, int n_slots, int n_hb, int chunk, int* slot, int* hb) {
  const int per_chunk = n_slots * chunk;
  const int full = (n_hb / chunk) * per_chunk;
  int c0, csize, rem;
  if (lin < full) { c0 = (lin / per_chunk) * chunk; csize = chunk; rem = lin % per_chunk; }
  else { c0 = (n_hb / chunk) * chunk; csize = n_hb - c0; rem = lin - full; }
  *slot = rem / csize;
  *hb = c0 + rem % csize;
}
static inline int chunk_for(long long bytes_per_hb, int n_hb, long long budget) {
  long long c = budget / (bytes_per_hb > 0 ? bytes_per_hb : 1);
  return (int)(c < 1 ? 1 : (c > n_hb ? n_hb : c));
}
