// Launch descriptors shared by the planner (host) and the kernels (device).
#pragma once
#include <cstdint>

namespace amap {

constexpr int kDevMaxLoops = 12;
constexpr int kDevMaxCons = 6;
constexpr int kMaxInputs = 24;
constexpr int kMaxOutputs = 8;
constexpr int kQuasiMaxDigits = 6;
constexpr int kStrip = 8;  // units per thread in the affine and strip kernels

// unsigned 32-bit division by an invariant divisor, multiply-and-shift form
// (Granlund & Montgomery 1994, "Division by invariant integers using
// multiplication", round-up variant): q = (t + ((n - t) >> sh1)) >> sh2 with
// t = mulhi(mul, n).
struct FastDiv {
  uint32_t mul, sh1, sh2, d;
};

struct DevCon {  // 0 <= off + sum coef[k] * i_k < extent   (all values fit 32 bits; the planner checks)
  int32_t off;
  int32_t extent;
  int32_t coef[kDevMaxLoops];
};

enum DevKind : int32_t { kDevAffine = 0, kDevTranspose = 1, kDevStrip = 2 };

// Transpose tiles: 8 chunks of 16 bytes of the destination-contiguous index a
// (128 bytes) by kTileB elements of the source-contiguous index b.
constexpr int kTileB = 128;
constexpr int kTileBytes = 16384;
constexpr int kTransposeThreads = 256;

// One piece of a composed map, ready to run.  Loops are in canonical order
// (destination stride descending).  All strides and offsets are in BYTES.
//
// Affine kernel: one item = one unit of `unit_bytes` bytes; the innermost loop
// counts units; ext/fd/sstride/dstride describe all loops.
//
// A quasi-affine piece (the composition of a reshape whose factors do not line
// up) runs on the affine kernel: beside the affine offsets it accumulates the
// inner form f and splits it into digits with multiply-and-shift divisions.
//
// Strip kernel: as the affine kernel, but loop `ku` (not the innermost) is cut
// into strips of kStrip iterations: ext[ku] counts strips, its strides and
// constraint coefficients are per strip, and one item = one strip of up to
// kStrip units that differ only in loop ku (ku_ext is that loop's true extent;
// ku_ss, ku_ds, ku_coef are its per-iteration strides and coefficients).
//
// Transpose kernel: ext/fd/sstride/dstride describe the BATCH loops only.  The
// tile indices are a (contiguous in the destination) and b (contiguous in the
// source); each may merge two loops of the piece: a = a_hi * a_in + a_lo with
// source offset a_lo * sa[0] + a_hi * sa[1] and destination offset a * es;
// b = b_hi * b_in + b_lo with destination offset b_lo * db[0] + b_hi * db[1]
// and source offset b * es.
struct DevPiece {
  int32_t kind;
  int32_t n_loops;
  int32_t input;  // slot of the source pointer, -1: fill only
  int32_t n_guards;
  int32_t n_domain;
  int32_t unit_bytes;
  int32_t prefetch;  // 1: ask L2 for the block's first source lines before waiting for the previous kernel
  int32_t out;  // slot of the destination pointer (0 unless the map has several outputs)
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
  // --- quasi-affine source (affine kernel only) -------------------------
  // qa_n > 0: the source offset is soff + sum_d qa_stride[d] * digit_d(f), f = qa_f0 + sum_k qa_fstride[k] * i_k
  // (in units, 32-bit wrap-around arithmetic), digits in the mixed radix qa_radix[] (innermost last).
  int32_t qa_n;
  uint32_t qa_f0;
  uint32_t qa_fstride[kDevMaxLoops];
  uint32_t qa_radix[kQuasiMaxDigits];
  FastDiv qa_fd[kQuasiMaxDigits];
  int64_t qa_stride[kQuasiMaxDigits];  // bytes
  // --- strip kernel only -----------------------------------------------
  int32_t ku;
  uint32_t ku_ext;
  int64_t ku_ss, ku_ds;
  int32_t ku_coef[kDevMaxCons];
  // --- transpose kernel only -------------------------------------------
  int32_t tr_unit;            // bytes per global access: 16, or less for pieces aligned to less; 0: shifted rows, -1: realigned source rows
  int32_t tile_ca;            // 16-byte kernel: 16-byte chunks of a per tile: 8 (by 128 elements of b), 4 (by 256), 16 (by 64), 32 (by 32)
  int64_t src_bytes;          // size of the source tensor (shifted-row kernel: guards the last aligned chunk)
  uint32_t ext_a, ext_b;      // merged extents, in elements
  uint32_t tiles_a, tiles_b;  // tiles along a / b
  uint32_t step_b;            // 16-byte kernel: elements of b between tiles (at most what a tile holds)
  uint32_t shift_wrap;        // shifted-row kernel: 1 when destination row b + 1 starts where row b ends
  FastDiv fd_tiles_a, fd_tiles_b;
  FastDiv fd_a_in, fd_b_in;  // inner extents of the merged indices
  int64_t sa[2];             // source byte strides of (a_lo, a_hi)
  int64_t db[2];             // destination byte strides of (b_lo, b_hi)
};

struct PtrTable {
  const char *src[kMaxInputs];
  char *dst0;                       // output 0: read at a fixed offset of the kernel parameters (the common case)
  char *dst_more[kMaxOutputs - 1];  // outputs 1.. of a map with several outputs
#ifdef __CUDACC__
  __host__ __device__ __forceinline__ char *dst(int out) const { return out == 0 ? dst0 : dst_more[out - 1]; }
#endif
  void set_dst(int out, char *p) {
    if (out == 0) dst0 = p;
    else dst_more[out - 1] = p;
  }
};

}  // namespace amap
