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

/* ---------------------------------------------------------------------------
 * Rows.  A consumer that walks the result row by row (rows x cols, row-major) need not decode every element from
 * scratch: when a row is the full range of the innermost loops of one piece, the loops OUTSIDE the row are decoded
 * once per row (amap_view_row_seek) and the loops INSIDE it are tabulated once per thread block
 * (amap_view_rows_build): a row is then `n_runs` runs of `run_len` consecutive source elements each, run j starting
 * at the row's base plus run_src[j], loaded if the row's constraint values plus run_con[j] pass the guards.  This is
 * what the strip kernel of the copy does per strip; an im2col row of 3x3 windows is nine runs of C elements.
 * ------------------------------------------------------------------------- */
#define AMAP_VIEW_MAX_RUNS 32

typedef struct amap_view_row_piece { /* one piece, 32-bit, outer loops and the table of a row's runs */
  int32_t n_outer;                   /* loops 0 .. n_outer-1 are outside a row                               */
  int32_t n_runs, run_len;           /* a row = n_runs runs of run_len elements                              */
  int32_t input, n_guards, n_domain;
  uint32_t b_s, b_l, fill_bits_lo, fill_bits_hi;
  uint32_t o_mul[AMAP_VIEW_MAX_LOOPS], o_ext[AMAP_VIEW_MAX_LOOPS], o_dst[AMAP_VIEW_MAX_LOOPS], o_src[AMAP_VIEW_MAX_LOOPS];
  uint8_t o_sh1[AMAP_VIEW_MAX_LOOPS], o_sh2[AMAP_VIEW_MAX_LOOPS];
  int32_t o_coef[AMAP_VIEW_MAX_LOOPS][AMAP_VIEW_MAX_CONS];
  int32_t c_off[AMAP_VIEW_MAX_CONS], c_ext[AMAP_VIEW_MAX_CONS];
  uint32_t run_src[AMAP_VIEW_MAX_RUNS];                    /* source offset of run j relative to the row's base */
  int32_t run_con[AMAP_VIEW_MAX_RUNS][AMAP_VIEW_MAX_CONS]; /* what run j adds to the constraint expressions      */
} amap_view_row_piece;

typedef struct amap_view_rows {
  int32_t usable; /* 0: some piece's rows are not whole runs (or the view is not `small`): use amap_view_locate */
  int32_t n_pieces;
  uint32_t cols;
  amap_view_row_piece piece[AMAP_VIEW_MAX_PIECES];
} amap_view_rows;

typedef struct amap_view_row_cursor {
  int32_t piece;                     /* the piece that holds the row, -1: none (cannot happen for a composed map) */
  uint32_t src_base;                 /* source element index contributed by the outer loops                       */
  int32_t con[AMAP_VIEW_MAX_CONS];   /* the constraint expressions at the row's first element                     */
} amap_view_row_cursor;

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

/* Tabulates piece p of the view for rows of `cols` elements into rows->piece[p] (any memory the caller's threads
 * share: call it from one thread per piece, then synchronise); clears rows->usable when the piece's rows are not
 * whole runs.  The caller sets rows->usable = v.small, rows->n_pieces and rows->cols beforehand. */
__host__ __device__ inline void amap_view_rows_build(const amap_device_view &v, int p, uint32_t cols, amap_view_rows *rows) {
  const amap_view_piece &pc = v.piece[p];
  amap_view_row_piece &rp = rows->piece[p];
  const int n = pc.n_loops, ng = pc.n_guards, nc = pc.n_guards + pc.n_domain;
  /* the loops inside a row: a dense suffix of the nest whose extents multiply to cols; the loop at its upper end
   * may lie partly inside: it is split, i = i_hi * split + i_lo, with i_lo inside the row */
  int first = n;
  int64_t span = 1, split = 0;
  while (first > 0 && span < (int64_t)cols && pc.dst_stride[first - 1] == span && span * pc.ext[first - 1] <= (int64_t)cols)
    span *= pc.ext[--first];
  if (span < (int64_t)cols && first > 0 && pc.dst_stride[first - 1] == span && (int64_t)cols % span == 0 &&
      pc.ext[first - 1] % ((int64_t)cols / span) == 0) {
    split = (int64_t)cols / span;
    span *= split;
  }
  bool ok = v.small && span == (int64_t)cols;
  /* the loops inside the row, outermost first: the inner part of a split loop, then loops first .. n-1 */
  int64_t in_ext[AMAP_VIEW_MAX_LOOPS + 1];
  int in_loop[AMAP_VIEW_MAX_LOOPS + 1];
  int n_in = 0;
  if (split) {
    in_ext[n_in] = split;
    in_loop[n_in++] = first - 1;
  }
  for (int k = first; k < n; ++k) {
    in_ext[n_in] = pc.ext[k];
    in_loop[n_in++] = k;
  }
  if (ok && n_in > 0) {  /* (no loop inside the row: cols = 1, every element a run of its own) */
    /* the innermost of them is the run: contiguous on both sides, no constraint looks at it */
    const int kr = in_loop[n_in - 1];
    ok = pc.dst_stride[kr] == 1 && (pc.input < 0 || pc.src_stride[kr] == 1);
    for (int c = 0; c < nc; ++c) ok = ok && pc.cons[c].coef[kr] == 0;
    /* a domain constraint that looks inside the row would hand parts of a row to another piece */
    for (int c = ng; c < nc; ++c)
      for (int q = 0; q < n_in; ++q) ok = ok && pc.cons[c].coef[in_loop[q]] == 0;
  }
  int64_t n_runs = 1;
  for (int q = 0; ok && q + 1 < n_in; ++q) n_runs *= in_ext[q];
  ok = ok && n_runs <= AMAP_VIEW_MAX_RUNS;
  if (!ok) {
    rows->usable = 0;
    return;
  }
  rp.n_outer = first;  /* loops 0 .. first-1; with a split the last of them counts i_hi */
  rp.n_runs = (int32_t)n_runs;
  rp.run_len = n_in > 0 ? (int32_t)in_ext[n_in - 1] : 1;
  rp.input = pc.input;
  rp.n_guards = ng;
  rp.n_domain = pc.n_domain;
  rp.b_s = (uint32_t)pc.b_s;
  rp.b_l = (uint32_t)pc.b_l;
  rp.fill_bits_lo = (uint32_t)pc.fill_bits;
  rp.fill_bits_hi = (uint32_t)(pc.fill_bits >> 32);
  for (int k = 0; k < first; ++k) {
    const uint32_t m = (split && k == first - 1) ? (uint32_t)split : 1u;  /* i_hi steps m iterations at a time */
    rp.o_ext[k] = (uint32_t)(pc.ext[k] / m);
    rp.o_dst[k] = (uint32_t)pc.dst_stride[k] * m;
    rp.o_src[k] = (uint32_t)pc.src_stride[k] * m;
    for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) rp.o_coef[k][c] = c < nc ? (int32_t)pc.cons[c].coef[k] * (int32_t)m : 0;
    if (m == 1) {
      rp.o_mul[k] = pc.fd_mul[k];
      rp.o_sh1[k] = pc.fd_sh1[k];
      rp.o_sh2[k] = pc.fd_sh2[k];
    } else {  /* division by o_dst[k]: multiply-and-shift, round-up form (Granlund & Montgomery 1994) */
      const uint32_t d = rp.o_dst[k];
      uint32_t l = 0;
      while (l < 32 && ((uint64_t)1 << l) < d) ++l;
      rp.o_mul[k] = (uint32_t)((((uint64_t)1 << 32) * (((uint64_t)1 << l) - d)) / d + 1);
      rp.o_sh1[k] = (uint8_t)(l < 1 ? l : 1);
      rp.o_sh2[k] = (uint8_t)(l > 0 ? l - 1 : 0);
    }
  }
  for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) {
    rp.c_off[c] = c < nc ? (int32_t)pc.cons[c].offset : 0;
    rp.c_ext[c] = c < nc ? (int32_t)pc.cons[c].extent : 1;
  }
  for (int j = 0; j < (int)n_runs; ++j) {  /* run j: its digits over the row's loops but the last, innermost last */
    uint32_t rem = (uint32_t)j, src = 0;
    int32_t con[AMAP_VIEW_MAX_CONS] = {0, 0, 0, 0};
    for (int q = n_in - 2; q >= 0; --q) {
      const uint32_t i = rem % (uint32_t)in_ext[q];
      rem /= (uint32_t)in_ext[q];
      src += i * (uint32_t)pc.src_stride[in_loop[q]];
      for (int c = 0; c < ng; ++c) con[c] += (int32_t)pc.cons[c].coef[in_loop[q]] * (int32_t)i;
    }
    rp.run_src[j] = src;
    for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) rp.run_con[j][c] = con[c];
  }
}

/* The row that starts at output element `row_start` (a multiple of rows.cols): finds its piece and decodes the
 * loops outside the row.  All values are 32-bit (the view is `small`). */
__host__ __device__ inline void amap_view_row_seek(const amap_view_rows &rows, uint32_t row_start, amap_view_row_cursor *cur) {
  cur->piece = -1;
  for (int p = 0; p < rows.n_pieces; ++p) {
    const amap_view_row_piece &rp = rows.piece[p];
    if (row_start < rp.b_s) continue;
    uint32_t rem = row_start - rp.b_s, s = rp.b_l;
    int32_t e[AMAP_VIEW_MAX_CONS];
    bool inside = true;
AMAP_PRAGMA_UNROLL
    for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] = rp.c_off[c];
AMAP_PRAGMA_UNROLL_1
    for (int k = 0; k < rp.n_outer; ++k) {
#ifdef __CUDA_ARCH__
      const uint32_t t = __umulhi(rp.o_mul[k], rem);
#else
      const uint32_t t = (uint32_t)(((uint64_t)rp.o_mul[k] * rem) >> 32);
#endif
      const uint32_t i = (t + ((rem - t) >> rp.o_sh1[k])) >> rp.o_sh2[k];
      inside = inside && i < rp.o_ext[k];
      rem -= i * rp.o_dst[k];
      s += i * rp.o_src[k];
AMAP_PRAGMA_UNROLL
      for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) e[c] += rp.o_coef[k][c] * (int32_t)i;
    }
    if (!inside || rem != 0) continue;
AMAP_PRAGMA_UNROLL
    for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c)
      if (c >= rp.n_guards && c < rp.n_guards + rp.n_domain) inside = inside && (uint32_t)e[c] < (uint32_t)rp.c_ext[c];
    if (!inside) continue;
    cur->piece = p;
    cur->src_base = s;
AMAP_PRAGMA_UNROLL
    for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c) cur->con[c] = e[c];
    return;
  }
}

/* Run j of the cursor's row: true and *src = the source element index of its first element if it is loaded, false if
 * its run_len elements are the piece's fill value. */
__host__ __device__ inline bool amap_view_row_run(const amap_view_row_piece &rp, const amap_view_row_cursor &cur, int j,
                                                  uint32_t *src) {
  bool load = rp.input >= 0;
AMAP_PRAGMA_UNROLL
  for (int c = 0; c < AMAP_VIEW_MAX_CONS; ++c)
    if (c < rp.n_guards) load = load && (uint32_t)(cur.con[c] + rp.run_con[j][c]) < (uint32_t)rp.c_ext[c];
  *src = cur.src_base + rp.run_src[j];
  return load;
}
#endif /* __CUDACC__ && !AMAP_DEVICE_STRUCTS_ONLY */

#endif /* AMAP_DEVICE_H_ */
