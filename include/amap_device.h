/*
 * amap_device.h -- reading THROUGH a composed map instead of running the copy.
 *
 * Section 2.2 of the paper wants the output of an operator to land where the
 * next operator needs it, so that no copy runs in between.  On a GPU the same
 * end is reached from the consumer's side: the kernel that would read the
 * result of a layout chain is handed the composed access map g' (Section 2.1,
 * equation (2)) and loads every element it wants straight from the external
 * input -- the "result" tensor never exists.
 *
 * amap_map_device_view() (amap.h) flattens a composed, single-stage,
 * single-output map into the plain struct below, small enough to be passed to
 * a kernel by value.  amap_view_locate() is the functor: output element index
 * -> (input, source element index) or the fill value.
 *
 * The header is plain C for the struct and CUDA C++ (under __CUDACC__, unless
 * AMAP_DEVICE_STRUCTS_ONLY is defined) for the device function; it has no
 * dependency on the library's internals.
 */
#ifndef AMAP_DEVICE_H_
#define AMAP_DEVICE_H_

#include <stdint.h>

#define AMAP_VIEW_MAX_PIECES 8
#define AMAP_VIEW_MAX_LOOPS 8
#define AMAP_VIEW_MAX_CONS 4

/* 0 <= offset + sum_k coef[k] * i_k < extent */
typedef struct amap_view_con {
  int64_t coef[AMAP_VIEW_MAX_LOOPS];
  int64_t offset, extent;
} amap_view_con;

/* One piece: out.flat[b_s + sum dst_stride[k] i_k] = in[input].flat[b_l + sum src_stride[k] i_k] over the box
 * 0 <= i_k < ext[k].  Loops are ordered by destination stride, largest first; destination strides are positive
 * and nested (each exceeds everything the loops after it can add up to), so an output index decodes into loop
 * indices digit by digit. */
typedef struct amap_view_piece {
  int32_t n_loops;
  int32_t input;    /* slot of the external input read, -1: the piece stores fill_bits */
  int32_t n_guards; /* cons[0 .. n_guards): where one fails the element is fill_bits   */
  int32_t n_domain; /* cons[n_guards .. n_guards + n_domain): where one fails the point is not this piece's */
  int64_t ext[AMAP_VIEW_MAX_LOOPS];
  int64_t dst_stride[AMAP_VIEW_MAX_LOOPS];
  int64_t src_stride[AMAP_VIEW_MAX_LOOPS];
  int64_t b_s, b_l;
  uint64_t fill_bits;
  amap_view_con cons[AMAP_VIEW_MAX_CONS];
  /* 32-bit fast path (amap_device_view.small): division by dst_stride[k] as multiply-and-shift,
   * q = (t + ((n - t) >> sh1)) >> sh2 with t = mulhi(mul, n)  (Granlund & Montgomery 1994, round-up form) */
  uint32_t fd_mul[AMAP_VIEW_MAX_LOOPS];
  uint8_t fd_sh1[AMAP_VIEW_MAX_LOOPS], fd_sh2[AMAP_VIEW_MAX_LOOPS];
} amap_view_piece;

typedef struct amap_device_view {
  int32_t n_pieces;
  int32_t elem_size;
  int32_t n_inputs;
  int32_t small;    /* 1: every index, offset and partial sum of the map fits 31 bits: amap_view_locate computes in
                       32-bit arithmetic with the precomputed divisions */
  int64_t out_numel;
  amap_view_piece piece[AMAP_VIEW_MAX_PIECES];
} amap_device_view;

/* where an output element comes from */
typedef struct amap_view_source {
  int32_t input;     /* slot of the external input, or -1: the element is `fill_bits` */
  int64_t index;     /* element index within that input (flat, row-major)             */
  int64_t run;       /* this and the next run-1 output elements come from consecutive source elements of the same
                        input (or are all fill): a consumer may fetch them with one vector load */
  uint64_t fill_bits;
} amap_view_source;

#if defined(__CUDACC__) && !defined(AMAP_DEVICE_STRUCTS_ONLY)
#ifdef __CUDA_ARCH__ /* unroll hints mean something to the device compiler only */
#define AMAP_PRAGMA_UNROLL _Pragma("unroll")
#define AMAP_PRAGMA_UNROLL_1 _Pragma("unroll 1")
#else
#define AMAP_PRAGMA_UNROLL
#define AMAP_PRAGMA_UNROLL_1
#endif
/* Output element `o` (0 <= o < out_numel) -> its source.  Returns false if no piece covers o (cannot happen for a
 * view made by amap_map_device_view: the pieces of a composed map cover the output exactly once).  One pass over the
 * piece's loops decodes the index digit by digit and accumulates the source offset and every constraint on the way,
 * so no per-loop value has to be kept. */
__host__ __device__ inline bool amap_view_locate(const amap_device_view &v, int64_t o, amap_view_source *out) {
  for (int p = 0; p < v.n_pieces; ++p) {
    const amap_view_piece &pc = v.piece[p];
    const int n = pc.n_loops, nc = pc.n_guards + pc.n_domain;
    bool inside = true, load = pc.input >= 0;
    int64_t s, left = 1;  /* left: elements of the innermost loop from this one on */
    if (o < pc.b_s) continue;
    if (v.small) {
      uint32_t rem = (uint32_t)(o - pc.b_s), s32 = (uint32_t)pc.b_l;
      int32_t e[AMAP_VIEW_MAX_CONS];
AMAP_PRAGMA_UNROLL
      for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] = c < nc ? (int32_t)pc.cons[c].offset : 0;
AMAP_PRAGMA_UNROLL_1
      for (int k = 0; k < n; ++k) {
#ifdef __CUDA_ARCH__
        const uint32_t t = __umulhi(pc.fd_mul[k], rem);
#else
        const uint32_t t = (uint32_t)(((uint64_t)pc.fd_mul[k] * rem) >> 32);
#endif
        const uint32_t i = (t + ((rem - t) >> pc.fd_sh1[k])) >> pc.fd_sh2[k];
        inside = inside && i < (uint32_t)pc.ext[k];
        rem -= i * (uint32_t)pc.dst_stride[k];
        s32 += i * (uint32_t)pc.src_stride[k];  /* wrap-around arithmetic: the true value fits 31 bits */
        if (nc > 0) {
AMAP_PRAGMA_UNROLL
          for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] += (int32_t)pc.cons[c].coef[k] * (int32_t)i;
        }
        if (k == n - 1) left = pc.ext[k] - (int64_t)i;
      }
      if (!inside || rem != 0) continue;
AMAP_PRAGMA_UNROLL
      for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) {
        if (c < nc) {
          const bool ok = (uint32_t)e[c] < (uint32_t)pc.cons[c].extent;
          if (c < pc.n_guards) load = load && ok;
          else inside = inside && ok;
        }
      }
      if (!inside) continue;
      s = (int64_t)s32;
    } else {
      int64_t rem = o - pc.b_s;
      int64_t e[AMAP_VIEW_MAX_CONS];
AMAP_PRAGMA_UNROLL
      for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] = c < nc ? pc.cons[c].offset : 0;
      s = pc.b_l;
AMAP_PRAGMA_UNROLL_1
      for (int k = 0; k < n; ++k) {
        const int64_t i = rem / pc.dst_stride[k];
        inside = inside && i < pc.ext[k];
        rem -= i * pc.dst_stride[k];
        s += i * pc.src_stride[k];
        if (nc > 0) {
AMAP_PRAGMA_UNROLL
          for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] += pc.cons[c].coef[k] * i;
        }
        if (k == n - 1) left = pc.ext[k] - i;
      }
      if (!inside || rem != 0) continue;
AMAP_PRAGMA_UNROLL
      for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) {
        if (c < nc) {
          const bool ok = e[c] >= 0 && e[c] < pc.cons[c].extent;
          if (c < pc.n_guards) load = load && ok;
          else inside = inside && ok;
        }
      }
      if (!inside) continue;
    }
    out->input = load ? pc.input : -1;
    out->index = load ? s : 0;
    out->fill_bits = pc.fill_bits;
    /* the innermost loop is a run when it is contiguous on both sides and no constraint looks at it */
    int64_t run = 1;
    if (n > 0) {
      const int in = n - 1;
      bool plain = pc.dst_stride[in] == 1 && (pc.input < 0 || pc.src_stride[in] == 1);
      for (int c = 0; c < nc && plain; ++c) plain = pc.cons[c].coef[in] == 0;
      if (plain) run = left;
    }
    out->run = run;
    return true;
  }
  return false;
}
#endif /* __CUDACC__ && !AMAP_DEVICE_STRUCTS_ONLY */

#endif /* AMAP_DEVICE_H_ */
