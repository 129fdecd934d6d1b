// Launch descriptors shared by the planner (host) and the kernels (device).
#pragma once
#include <cstdint>

namespace amap {

constexpr int kDevMaxLoops = 12;
constexpr int kDevMaxCons = 6;
constexpr int kMaxInputs = 24;

// unsigned 32-bit division by an invariant divisor, multiply-and-shift form
// (Granlund & Montgomery 1994, "Division by invariant integers using
// multiplication", round-up variant): q = (t + ((n - t) >> sh1)) >> sh2 with
// t = mulhi(mul, n).
struct FastDiv {
  uint32_t mul, sh1, sh2, d;
};

struct DevCon {  // 0 <= off + sum coef[k] * i_k < extent
  int64_t off;
  int64_t extent;
  int32_t coef[kDevMaxLoops];
};

enum DevKind : int32_t { kDevAffine = 0, kDevTranspose = 1 };

// One piece of a composed map, ready to run.  Loops are in canonical order
// (destination stride descending).  For the affine kernel one "item" is one
// unit of `unit_bytes` bytes; the innermost loop counts units and all strides
// and offsets are in BYTES.
struct DevPiece {
  int32_t kind;
  int32_t n_loops;
  int32_t input;  // slot of the source pointer, -1: fill only
  int32_t n_guards;
  int32_t n_domain;
  int32_t unit_bytes;
  uint32_t first_block;  // first block of this piece inside its launch
  uint32_t n_blocks;
  uint64_t n_items;
  uint64_t fill[2];  // the fill pattern replicated over 16 bytes
  int64_t soff, doff;
  uint32_t ext[kDevMaxLoops];
  FastDiv fd[kDevMaxLoops];
  int64_t sstride[kDevMaxLoops];
  int64_t dstride[kDevMaxLoops];
  DevCon cons[kDevMaxCons];  // guards first, then domain constraints
  // --- transpose kernel only -------------------------------------------
  // Tile = TA elements of loop `la` (destination-contiguous) x TB elements of
  // loop `lb` (source-contiguous); the remaining loops are the batch.
  int32_t la, lb;
  uint32_t tiles_a, tiles_b;  // tiles along la / lb
  FastDiv fd_tiles_a, fd_tiles_b;
  int32_t pad_[2];
};

struct PtrTable {
  const char *src[kMaxInputs];
  char *dst;
};

}  // namespace amap
