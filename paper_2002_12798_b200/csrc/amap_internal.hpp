// Internal data model of the host algebra (not part of the C ABI).
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "amap.h"

#include <cstdlib>

namespace amap {

// AMAP_LOG set to anything but "" or "0": print composed pieces and failures to stderr
inline bool log_enabled() {
  const char *v = getenv("AMAP_LOG");
  return v != nullptr && v[0] != '\0' && !(v[0] == '0' && v[1] == '\0');
}

// c0 + sum_k c[k] * i_k over a piece's loops
struct Aff {
  int64_t c0 = 0;
  std::vector<int64_t> c;
};

// 0 <= e < extent
struct Con {
  Aff e;
  int64_t extent = 0;
};

// A source offset that is only QUASI-affine in the loops (the reverse of a store composed with a reshape whose
// factors do not line up needs floor-division and remainder; the paper leaves these to ISL, Section 2.1): the
// affine form f(i) is an offset into a tensor that was composed away, and the source offset is
//     srcoff.c0 + sum_k stride[k] * digit_k(f),
// digit_k being f's digits in the mixed radix (radix[0], ..., radix[K-1]), innermost last -- the loop indices of the
// statement that wrote that tensor.
struct QuasiSrc {
  bool on = false;
  Aff f;
  std::vector<int64_t> radix, stride;
};

// One loop nest of the composed form: for i in the box (and where `domain`
// holds) dst.flat[dst(i)] = guards hold ? src.flat[srcoff(i)] : fill.
struct Piece {
  std::vector<int64_t> ext;
  Aff dst;
  int src = AMAP_CONST;  // tensor id while composing; input slot in a finished map
  Aff srcoff;
  QuasiSrc qa;  // when on, srcoff holds the constant only
  std::vector<Con> guards;
  std::vector<Con> domain;
  uint64_t fill = 0;
  int out = 0;  // which output of the map the piece writes (final stage of a map with several outputs)
  int n() const { return (int)ext.size(); }
};

struct TensorInfo {
  std::vector<int64_t> shape;
  std::vector<int64_t> stride;  // row-major, elements
  int64_t numel = 0;
  int input_slot = -1;  // >= 0 for external inputs
};

struct Status {
  int code = AMAP_OK;
  std::string msg;
  bool ok() const { return code == AMAP_OK; }
};

// ---- simplify.cpp --------------------------------------------------------
// interval of an affine expression over the box [0,ext)
void aff_range(const Aff &a, const std::vector<int64_t> &ext, int64_t *lo, int64_t *hi);
// Drops constraints that always hold, clips single-loop domain constraints
// into the box.  Returns false when the piece has no points left.
bool tighten(Piece &p);
// number of loop points of the piece (box and domain); -1 if it cannot be counted cheaply
int64_t count_points(const Piece &p);
void reverse_loop(Piece &p, int k);
void permute_loops(Piece &p, const std::vector<int> &order);
void drop_unit_loops(Piece &p);
// final canonical form of a composed map's pieces (splits single-loop guards
// into copy + fill pieces, sorts by destination stride, merges loops)
Status canonicalise(std::vector<Piece> &pieces);

// elements of the contiguous run (on both sides) that loop `in` of the piece walks, as a power of two that divides
// everything a vector access needs divided: 1 when the loop is no run
int64_t piece_run_elems(const Piece &p, int in, int64_t cap);

// ---- compose.cpp ---------------------------------------------------------
// A composed map runs as one or more STAGES.  Normally there is one: every intermediate tensor was composed
// away.  An intermediate that could not be composed affinely (or, on request, every intermediate) is kept as a
// temporary: an earlier stage writes it, later stages read it like an input (piece.src = n_inputs + temporary).
struct StageInfo {
  int first_piece = 0, n_pieces = 0;
  int dst_temp = -1;  // -1: the stage writes the output(s): every piece names its output in Piece::out
  int64_t numel = 0;  // elements of the temporary written; of output 0 for the final stage
};

struct Map {
  int elem_size = 0;
  std::vector<int64_t> in_numel;
  int64_t out_numel = 0;             // output 0
  std::vector<int64_t> out_numels;   // every output
  std::vector<int64_t> temp_numel;
  std::vector<StageInfo> stages;
  std::vector<Piece> pieces;  // all stages, in execution order
  // storage for the C views handed out by amap_map_get_piece
  std::vector<std::vector<amap_constraint>> guard_views, domain_views;
};

}  // namespace amap

struct amap_map {
  amap::Map m;
};
