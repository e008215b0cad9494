// Tile propagation through chains of reshape / permute operators and the composed, strength-reduced tile map
// (the paper's section 4.3).  Host code only.
//
// Representation: the tensor's index space is a mixed-radix number whose digits ("atoms") are factors of the
// source dimensions.  A reshape regroups adjacent atoms (splitting one where a new boundary falls inside it), a
// permute reorders groups.  Two atoms are special: the innermost tile_w columns of the last source dimension and the
// innermost tile_h rows of the one before it.  Together they are one tile's interior; a chain is legal when it never
// cuts them and leaves them as the innermost factors of the destination's column and row axes.  All other atoms are
// digits of the tile number, and the tile map is "read the source digits, weight them by their destination
// strides".
#include <new>
#include <vector>

#include "fbl_internal.h"

namespace {

enum Role { TILE_DIGIT = 0, INTRA_ROW = 1, INTRA_COL = 2 };
struct Atom { int64_t size; int role; };

struct State {
  std::vector<Atom> atoms;                    // by id
  std::vector<int> src_order;                 // atom ids, outermost first, in the source's flattening order
  std::vector<std::vector<int>> dims;         // current dimensions, each a list of atom ids, outermost first
};

// Replace atom `id` by (outer, inner) with outer * inner = its size; both keep its place in every ordering.
int split_atom(State& s, int id, int64_t outer) {
  const int64_t inner = s.atoms[id].size / outer;
  const int role = s.atoms[id].role;
  s.atoms[id].size = outer;
  s.atoms.push_back({inner, role});
  const int nid = (int)s.atoms.size() - 1;
  for (size_t i = 0; i < s.src_order.size(); ++i)
    if (s.src_order[i] == id) { s.src_order.insert(s.src_order.begin() + i + 1, nid); break; }
  for (auto& d : s.dims)
    for (size_t i = 0; i < d.size(); ++i)
      if (d[i] == id) { d.insert(d.begin() + i + 1, nid); return nid; }
  return nid;
}

// Which check the current arrangement fails (FBL_TP_OK: tiles are intact and in place).
int check_state(const State& s) {
  if (s.dims.empty()) return FBL_TP_DIMENSION;
  const int last = (int)s.dims.size() - 1;
  for (int role : {INTRA_COL, INTRA_ROW}) {
    int where = -1, pos = -1, id = -1;
    for (int d = 0; d <= last; ++d)
      for (size_t i = 0; i < s.dims[d].size(); ++i)
        if (s.atoms[s.dims[d][i]].role == role && s.atoms[s.dims[d][i]].size > 1) { where = d; pos = (int)i; id = s.dims[d][i]; }
    if (id < 0) continue;                                    // tile extent 1 along this axis: nothing to preserve
    if (role == INTRA_COL) {
      if (where != last) return FBL_TP_DIMENSION;            // the tile's column axis left the column axis
      if (pos != (int)s.dims[last].size() - 1) return FBL_TP_CONTINUITY;     // no longer stride-1
    } else {
      if (where == last) return FBL_TP_DIMENSION;            // the tile's row axis became (part of) the column axis
      // it must be the innermost factor of the whole row space: nothing non-trivial after it among the row dims
      bool after = false;
      for (int d = where; d < last; ++d)
        for (size_t i = (d == where ? (size_t)pos + 1 : 0); i < s.dims[d].size(); ++i)
          if (s.atoms[s.dims[d][i]].size > 1) after = true;
      if (after) return FBL_TP_CONTINUITY;
    }
  }
  return FBL_TP_OK;
}

}  // namespace

struct fbl_tile_chain {
  std::vector<fbl_tile_term> terms;
  int64_t tiles;
};

extern "C" {

int fbl_tile_chain_create(const int64_t* shape, int rank, int tile_h, int tile_w, const fbl_view_op* ops, int n_ops,
                          fbl_tile_chain** out, int32_t* failed_op, int32_t* failed_check) {
  if (!shape || !out || rank < 2 || rank > 8 || tile_h < 1 || tile_w < 1 || n_ops < 0 || (n_ops > 0 && !ops)) return FBL_ERR_INVALID_ARG;
  *out = nullptr;
  auto fail = [&](int op, int check) {
    if (failed_op) *failed_op = op;
    if (failed_check) *failed_check = check;
    return (int)FBL_ERR_UNSUPPORTED_SHAPE;
  };
  if (failed_op) *failed_op = -1;
  if (failed_check) *failed_check = FBL_TP_OK;
  State s;
  int64_t total = 1;
  for (int d = 0; d < rank; ++d) {
    if (shape[d] <= 0) return FBL_ERR_INVALID_ARG;
    total *= shape[d];
    s.atoms.push_back({shape[d], TILE_DIGIT});
    s.src_order.push_back(d);
    s.dims.push_back({d});
  }
  // the source's own tiling: whole tiles along both axes (op index -1: the layout itself is illegal for this tile)
  if (shape[rank - 1] % tile_w != 0 || shape[rank - 2] % tile_h != 0) return fail(-1, FBL_TP_BOUNDARY);
  if (tile_w > 1) { const int in = split_atom(s, rank - 1, shape[rank - 1] / tile_w); s.atoms[in].role = INTRA_COL; }
  if (tile_h > 1) { const int in = split_atom(s, rank - 2, shape[rank - 2] / tile_h); s.atoms[in].role = INTRA_ROW; }
  const int64_t tiles = total / ((int64_t)tile_h * tile_w);

  int first_bad = -2;                       // first operator of the trailing run of illegal arrangements
  for (int k = 0; k < n_ops; ++k) {
    const fbl_view_op& op = ops[k];
    if (op.rank < 1 || op.rank > 8) return FBL_ERR_INVALID_ARG;
    if (op.kind == FBL_VIEW_EXPAND) return fail(k, FBL_TP_DIMENSION);      // element count changes: tile granularity is lost
    if (op.kind == FBL_VIEW_PERMUTE) {
      if (op.rank != (int)s.dims.size()) return FBL_ERR_INVALID_ARG;
      std::vector<std::vector<int>> nd(op.rank);
      std::vector<char> seen(op.rank, 0);
      for (int a = 0; a < op.rank; ++a) {
        if (op.perm[a] < 0 || op.perm[a] >= op.rank || seen[op.perm[a]]) return FBL_ERR_INVALID_ARG;
        seen[op.perm[a]] = 1;
        nd[a] = s.dims[op.perm[a]];
      }
      s.dims.swap(nd);
    } else if (op.kind == FBL_VIEW_RESHAPE) {
      int64_t nt = 1;
      for (int a = 0; a < op.rank; ++a) { if (op.shape[a] <= 0) return FBL_ERR_INVALID_ARG; nt *= op.shape[a]; }
      if (nt != total) return fail(k, FBL_TP_DIMENSION);
      std::vector<int> flat;
      for (auto& d : s.dims) for (int id : d) flat.push_back(id);
      s.dims.assign(1, flat);                // one group; split_atom keeps it consistent while we cut it up
      std::vector<std::vector<int>> nd(op.rank);
      size_t cur = 0;
      for (int a = 0; a < op.rank; ++a) {
        int64_t acc = 1;
        const int64_t target = op.shape[a];
        while (acc < target) {
          if (cur >= s.dims[0].size()) return fail(k, FBL_TP_BOUNDARY);
          const int id = s.dims[0][cur];
          const int64_t sz = s.atoms[id].size;
          if (target % (acc * sz) == 0) { nd[a].push_back(id); acc *= sz; ++cur; continue; }
          const int64_t need = target / acc;               // the new boundary falls inside this atom
          if (sz % need != 0) return fail(k, FBL_TP_BOUNDARY);
          if (s.atoms[id].role != TILE_DIGIT) return fail(k, FBL_TP_BOUNDARY);      // it would cut a tile
          split_atom(s, id, need);
          nd[a].push_back(id); acc *= need; ++cur;
        }
        // size-1 atoms that follow belong anywhere; leave them for the next dimension
      }
      for (; cur < s.dims[0].size(); ++cur) nd[op.rank - 1].push_back(s.dims[0][cur]);     // trailing size-1 atoms
      s.dims.swap(nd);
    } else {
      return FBL_ERR_INVALID_ARG;
    }
    const int c = check_state(s);
    if (c == FBL_TP_OK) first_bad = -2;
    else if (first_bad == -2) first_bad = k;
  }
  const int final_check = check_state(s);
  if (final_check != FBL_TP_OK) return fail(first_bad == -2 ? n_ops - 1 : first_bad, final_check);

  // tile digits in source order with their strides in the source and destination tile numbering
  std::vector<int> digits;
  for (int id : s.src_order) if (s.atoms[id].role == TILE_DIGIT && s.atoms[id].size > 1) digits.push_back(id);
  std::vector<int64_t> sstride(s.atoms.size(), 0), dstride(s.atoms.size(), 0);
  int64_t st = 1;
  for (int i = (int)digits.size() - 1; i >= 0; --i) { sstride[digits[i]] = st; st *= s.atoms[digits[i]].size; }
  st = 1;
  for (int d = (int)s.dims.size() - 1; d >= 0; --d)
    for (int i = (int)s.dims[d].size() - 1; i >= 0; --i) {
      const int id = s.dims[d][i];
      if (s.atoms[id].role == TILE_DIGIT && s.atoms[id].size > 1) { dstride[id] = st; st *= s.atoms[id].size; }
    }
  fbl_tile_chain* c = new (std::nothrow) fbl_tile_chain();
  if (!c) return FBL_ERR_INVALID_ARG;
  c->tiles = tiles;
  // strength reduction: neighbouring source digits whose destination strides are also those of neighbours collapse
  // into one digit ((j / s) % (a b) replaces two divisions and two modulos); the outermost digit needs no modulo
  for (size_t i = 0; i < digits.size();) {
    int64_t size = s.atoms[digits[i]].size;
    size_t jn = i;
    while (jn + 1 < digits.size() &&
           dstride[digits[jn]] == dstride[digits[jn + 1]] * s.atoms[digits[jn + 1]].size) {
      ++jn;
      size *= s.atoms[digits[jn]].size;
    }
    c->terms.push_back({sstride[digits[jn]], i == 0 ? 0 : size, dstride[digits[jn]]});
    i = jn + 1;
  }
  *out = c;
  return FBL_OK;
}

void fbl_tile_chain_destroy(fbl_tile_chain* chain) { delete chain; }

int64_t fbl_tile_chain_tiles(const fbl_tile_chain* chain) { return chain ? chain->tiles : -1; }

int fbl_tile_chain_terms(const fbl_tile_chain* chain, fbl_tile_term* terms, int max_terms) {
  if (!chain || (max_terms > 0 && !terms)) return FBL_ERR_INVALID_ARG;
  const int n = (int)chain->terms.size();
  for (int i = 0; i < n && i < max_terms; ++i) terms[i] = chain->terms[i];
  return n;
}

int fbl_tile_chain_map(const fbl_tile_chain* chain, int64_t src_tile, int64_t* dst_tile) {
  if (!chain || !dst_tile || src_tile < 0 || src_tile >= chain->tiles) return FBL_ERR_INVALID_ARG;
  int64_t i = 0;
  for (const fbl_tile_term& t : chain->terms) {
    int64_t digit = src_tile / t.div;
    if (t.mod) digit %= t.mod;
    i += digit * t.mul;
  }
  *dst_tile = i;
  return FBL_OK;
}

}  // extern "C"
