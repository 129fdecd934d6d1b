/*
 * layout_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow CPU restatement of the layout operators whose load/store loop
 * nests the paper's data-movement elimination composes (Section 2, equations
 * (load) and (store); Section 2.1 names the operator families).  Every operator
 * here is executed by itself as a naive loop nest over its OUTPUT index and
 * writes a fully materialised result: nothing is ever composed, reordered,
 * tiled or fused.  Running a chain means calling these one after another with
 * one intermediate buffer per operator, which is exactly the program that the
 * paper's rewrite (Section 2.1, equations (1) and (2)) must leave unchanged
 * for every reader.
 *
 * This file shares no code with the CUDA library and is used only by the test
 * suite, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Elements are opaque patterns of `es` bytes (no floating-point arithmetic
 * happens anywhere), tensors are dense and row-major, and all indices are
 * int64_t.  Every function returns 0 on success and a negative number for an
 * argument it refuses.  `nt` is the number of OpenMP threads over the
 * outermost output dimension (1 = serial); the loop bodies are the same.
 *
 * Pins: tests/test_oracle_pins.py (closed forms, bijection and involution
 * properties, library special cases, brute force).  No function in this file
 * is "parity unpinned".
 */
#include <stdint.h>
#include <string.h>
#include <stdlib.h>

#define ORACLE_MAX_RANK 8
#define ORACLE_MAX_LOOPS 12

static int64_t numel(int rank, const int64_t *shape) {
  int64_t n = 1;
  for (int d = 0; d < rank; ++d) n *= shape[d];
  return n;
}

/* flat row-major offset of a multi-index */
static int64_t flat_of(int rank, const int64_t *shape, const int64_t *idx) {
  int64_t f = 0;
  for (int d = 0; d < rank; ++d) f = f * shape[d] + idx[d];
  return f;
}

/* advance idx[first..rank) like an odometer; returns 0 when it wraps around */
static int next_index(int first, int rank, const int64_t *shape, int64_t *idx) {
  for (int d = rank - 1; d >= first; --d) {
    if (++idx[d] < shape[d]) return 1;
    idx[d] = 0;
  }
  return 0;
}

static void copy_elem(unsigned char *dst, int64_t o, const unsigned char *src, int64_t i, int es) {
  memcpy(dst + o * es, src + i * es, (size_t)es);
}

static int bad_common(int rank, const int64_t *shape, int es) {
  if (rank < 1 || rank > ORACLE_MAX_RANK || !shape) return 1;
  if (!(es == 1 || es == 2 || es == 4 || es == 8 || es == 16)) return 1;
  for (int d = 0; d < rank; ++d)
    if (shape[d] < 0) return 1;
  return 0;
}

/* reshape: the flat buffer is unchanged (Section 2.1 lists it among the pure
 * copies); out.flat[k] = in.flat[k]. */
int oracle_reshape(const void *in, void *out, int in_rank, const int64_t *in_shape, int out_rank,
                   const int64_t *out_shape, int es, int nt) {
  (void)nt;
  if (bad_common(in_rank, in_shape, es) || bad_common(out_rank, out_shape, es)) return -1;
  int64_t n = numel(in_rank, in_shape);
  if (n != numel(out_rank, out_shape)) return -2;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
  for (int64_t k = 0; k < n; ++k) copy_elem(dst, k, src, k, es);
  return 0;
}

/* transpose(perm): out.shape[d] = in.shape[perm[d]] and
 * out[o] = in[j] with j[perm[d]] = o[d]. */
int oracle_transpose(const void *in, void *out, int rank, const int64_t *in_shape, const int32_t *perm,
                     int es, int nt) {
  if (bad_common(rank, in_shape, es) || !perm) return -1;
  int seen[ORACLE_MAX_RANK] = {0};
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) {
    if (perm[d] < 0 || perm[d] >= rank || seen[perm[d]]) return -2;
    seen[perm[d]] = 1;
    out_shape[d] = in_shape[perm[d]];
  }
  if (numel(rank, in_shape) == 0) return 0;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t o0 = 0; o0 < out_shape[0]; ++o0) {
    int64_t o[ORACLE_MAX_RANK] = {0}, j[ORACLE_MAX_RANK];
    o[0] = o0;
    do {
      for (int d = 0; d < rank; ++d) j[perm[d]] = o[d];
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, j), es);
    } while (next_index(1, rank, out_shape, o));
  }
  return 0;
}

/* strided slice, step >= 1: out.shape[d] = ceil((stop-start)/step),
 * out[o] = in[start + step*o]. */
int oracle_slice(const void *in, void *out, int rank, const int64_t *in_shape, const int64_t *start,
                 const int64_t *stop, const int64_t *step, int es, int nt) {
  if (bad_common(rank, in_shape, es) || !start || !stop || !step) return -1;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) {
    if (step[d] < 1 || start[d] < 0 || stop[d] > in_shape[d] || stop[d] < start[d]) return -2;
    out_shape[d] = (stop[d] - start[d] + step[d] - 1) / step[d];
  }
  if (numel(rank, out_shape) == 0) return 0;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t o0 = 0; o0 < out_shape[0]; ++o0) {
    int64_t o[ORACLE_MAX_RANK] = {0}, j[ORACLE_MAX_RANK];
    o[0] = o0;
    do {
      for (int d = 0; d < rank; ++d) j[d] = start[d] + step[d] * o[d];
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, j), es);
    } while (next_index(1, rank, out_shape, o));
  }
  return 0;
}

/* concat on `axis`: out[..., off_q + a, ...] = in_q[..., a, ...], off_q the
 * running sum of the inputs' extents on that axis.  `in_axis_extent[q]` is
 * in_q.shape[axis]; `other_shape` gives the shape shared by all inputs (its
 * entry at `axis` is ignored). */
int oracle_concat(int n_in, const void *const *ins, const int64_t *in_axis_extent, void *out, int rank,
                  const int64_t *other_shape, int axis, int es, int nt) {
  if (bad_common(rank, other_shape, es) || n_in < 1 || !ins || !in_axis_extent) return -1;
  if (axis < 0 || axis >= rank) return -2;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) out_shape[d] = other_shape[d];
  out_shape[axis] = 0;
  for (int q = 0; q < n_in; ++q) {
    if (in_axis_extent[q] < 0) return -2;
    out_shape[axis] += in_axis_extent[q];
  }
  unsigned char *dst = (unsigned char *)out;
  int64_t off = 0;
  for (int q = 0; q < n_in; ++q) {
    int64_t in_shape[ORACLE_MAX_RANK];
    for (int d = 0; d < rank; ++d) in_shape[d] = other_shape[d];
    in_shape[axis] = in_axis_extent[q];
    const unsigned char *src = (const unsigned char *)ins[q];
    if (numel(rank, in_shape) > 0) {
#pragma omp parallel for num_threads(nt) schedule(static)
      for (int64_t a0 = 0; a0 < in_shape[0]; ++a0) {
        int64_t a[ORACLE_MAX_RANK] = {0}, o[ORACLE_MAX_RANK];
        a[0] = a0;
        do {
          for (int d = 0; d < rank; ++d) o[d] = a[d];
          o[axis] = off + a[axis];
          copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, a), es);
        } while (next_index(1, rank, in_shape, a));
      }
    }
    off += in_axis_extent[q];
  }
  return 0;
}

/* constant-zero pad: out is all-zero bits, then out[o + lo] = in[o]. */
int oracle_pad(const void *in, void *out, int rank, const int64_t *in_shape, const int64_t *lo,
               const int64_t *hi, int es, int nt) {
  if (bad_common(rank, in_shape, es) || !lo || !hi) return -1;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) {
    if (lo[d] < 0 || hi[d] < 0) return -2;
    out_shape[d] = lo[d] + in_shape[d] + hi[d];
  }
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
  memset(dst, 0, (size_t)(numel(rank, out_shape) * es));
  if (numel(rank, in_shape) == 0) return 0;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t a0 = 0; a0 < in_shape[0]; ++a0) {
    int64_t a[ORACLE_MAX_RANK] = {0}, o[ORACLE_MAX_RANK];
    a[0] = a0;
    do {
      for (int d = 0; d < rank; ++d) o[d] = a[d] + lo[d];
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, a), es);
    } while (next_index(1, rank, in_shape, a));
  }
  return 0;
}

/* im2col window gather from an ALREADY PADDED NHWC tensor [N,Hp,Wp,C]
 * (a non-injective load: one input element feeds up to kh*kw outputs):
 *   out[(n*Ho+ho)*Wo+wo, (r*kw+s)*C+c] = in[n, ho*stride+r, wo*stride+s, c],
 *   Ho = (Hp-kh)/stride+1, Wo = (Wp-kw)/stride+1.
 * The zero border comes from oracle_pad, run as its own operator before. */
int oracle_window_gather(const void *in, void *out, const int64_t *in_shape /* N,Hp,Wp,C */, int64_t kh,
                         int64_t kw, int64_t stride, int es, int nt) {
  if (bad_common(4, in_shape, es) || kh < 1 || kw < 1 || stride < 1) return -1;
  const int64_t N = in_shape[0], Hp = in_shape[1], Wp = in_shape[2], C = in_shape[3];
  if (Hp < kh || Wp < kw) return -2;
  const int64_t Ho = (Hp - kh) / stride + 1, Wo = (Wp - kw) / stride + 1;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t ho = 0; ho < Ho; ++ho)
      for (int64_t wo = 0; wo < Wo; ++wo)
        for (int64_t r = 0; r < kh; ++r)
          for (int64_t s = 0; s < kw; ++s)
            for (int64_t c = 0; c < C; ++c) {
              int64_t row = (n * Ho + ho) * Wo + wo;
              int64_t col = (r * kw + s) * C + c;
              int64_t i = ((n * Hp + (ho * stride + r)) * Wp + (wo * stride + s)) * C + c;
              copy_elem(dst, row * (kh * kw * C) + col, src, i, es);
            }
  return 0;
}

/* The window gather with dilated taps and a choice of column order (the im2col families of the common
 * frameworks; the paper's Section 2.1 treats all of them as load/store pairs with a non-injective load):
 *   tap (r, s) of output pixel (ho, wo) reads in[n, ho*stride + r*dilation, wo*stride + s*dilation, c],
 *   Ho = (Hp - dilation*(kh-1) - 1)/stride + 1, likewise Wo,
 *   column = (r*kw + s)*C + c   when crs_order == 0  (channel fastest, NHWC style),
 *   column = (c*kh + r)*kw + s  when crs_order != 0  (tap fastest, NCHW style).
 * The zero border comes from oracle_pad, run as its own operator before. */
int oracle_window_gather_ex(const void *in, void *out, const int64_t *in_shape /* N,Hp,Wp,C */, int64_t kh,
                            int64_t kw, int64_t stride, int64_t dilation, int crs_order, int es, int nt) {
  if (bad_common(4, in_shape, es) || kh < 1 || kw < 1 || stride < 1 || dilation < 1) return -1;
  const int64_t N = in_shape[0], Hp = in_shape[1], Wp = in_shape[2], C = in_shape[3];
  const int64_t span_h = dilation * (kh - 1) + 1, span_w = dilation * (kw - 1) + 1;
  if (Hp < span_h || Wp < span_w) return -2;
  const int64_t Ho = (Hp - span_h) / stride + 1, Wo = (Wp - span_w) / stride + 1;
  const int64_t cols = kh * kw * C;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t ho = 0; ho < Ho; ++ho)
      for (int64_t wo = 0; wo < Wo; ++wo)
        for (int64_t r = 0; r < kh; ++r)
          for (int64_t s = 0; s < kw; ++s)
            for (int64_t c = 0; c < C; ++c) {
              int64_t row = (n * Ho + ho) * Wo + wo;
              int64_t col = crs_order ? (c * kh + r) * kw + s : (r * kw + s) * C + c;
              int64_t h = ho * stride + r * dilation, w = wo * stride + s * dilation;
              copy_elem(dst, row * cols + col, src, ((n * Hp + h) * Wp + w) * C + c, es);
            }
  return 0;
}

/* tile(reps): the whole tensor laid side by side reps[d] times along every
 * axis (Section 2.1 names tile and repeat among the pure copies):
 * out.shape[d] = reps[d]*in.shape[d], out[o] = in[j] with j[d] = o[d] mod in.shape[d]. */
int oracle_tile(const void *in, void *out, int rank, const int64_t *in_shape, const int64_t *reps, int es,
                int nt) {
  if (bad_common(rank, in_shape, es) || !reps) return -1;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) {
    if (reps[d] < 1) return -2;
    out_shape[d] = reps[d] * in_shape[d];
  }
  if (numel(rank, in_shape) == 0) return 0;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t o0 = 0; o0 < out_shape[0]; ++o0) {
    int64_t o[ORACLE_MAX_RANK] = {0}, j[ORACLE_MAX_RANK];
    o[0] = o0;
    do {
      for (int d = 0; d < rank; ++d) j[d] = o[d] % in_shape[d];
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, j), es);
    } while (next_index(1, rank, out_shape, o));
  }
  return 0;
}

/* repeat(axis, count): every element count times in a row along one axis:
 * out.shape[axis] = count*in.shape[axis], out[o] = in[j] with
 * j[axis] = o[axis] div count and j[d] = o[d] elsewhere. */
int oracle_repeat(const void *in, void *out, int rank, const int64_t *in_shape, int axis, int64_t count,
                  int es, int nt) {
  if (bad_common(rank, in_shape, es) || axis < 0 || axis >= rank || count < 1) return -1;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) out_shape[d] = in_shape[d];
  out_shape[axis] = count * in_shape[axis];
  if (numel(rank, in_shape) == 0) return 0;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t o0 = 0; o0 < out_shape[0]; ++o0) {
    int64_t o[ORACLE_MAX_RANK] = {0}, j[ORACLE_MAX_RANK];
    o[0] = o0;
    do {
      for (int d = 0; d < rank; ++d) j[d] = o[d];
      j[axis] = o[axis] / count;
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, j), es);
    } while (next_index(1, rank, out_shape, o));
  }
  return 0;
}

/* split(axis, sizes): the tensor cut into consecutive parts along one axis;
 * this writes part `part`: out.shape[axis] = sizes[part],
 * out[o] = in[j] with j[axis] = o[axis] + sizes[0] + ... + sizes[part-1].
 * The sizes must add up to in.shape[axis]. */
int oracle_split_part(const void *in, void *out, int rank, const int64_t *in_shape, int axis, int n_parts,
                      const int64_t *sizes, int part, int es, int nt) {
  if (bad_common(rank, in_shape, es) || axis < 0 || axis >= rank || n_parts < 1 || !sizes || part < 0 ||
      part >= n_parts)
    return -1;
  int64_t total = 0, first = 0;
  for (int q = 0; q < n_parts; ++q) {
    if (sizes[q] < 0) return -2;
    if (q < part) first += sizes[q];
    total += sizes[q];
  }
  if (total != in_shape[axis]) return -2;
  int64_t out_shape[ORACLE_MAX_RANK];
  for (int d = 0; d < rank; ++d) out_shape[d] = in_shape[d];
  out_shape[axis] = sizes[part];
  if (numel(rank, out_shape) == 0) return 0;
  const unsigned char *src = (const unsigned char *)in;
  unsigned char *dst = (unsigned char *)out;
#pragma omp parallel for num_threads(nt) schedule(static)
  for (int64_t o0 = 0; o0 < out_shape[0]; ++o0) {
    int64_t o[ORACLE_MAX_RANK] = {0}, j[ORACLE_MAX_RANK];
    o[0] = o0;
    do {
      for (int d = 0; d < rank; ++d) j[d] = o[d];
      j[axis] = o[axis] + first;
      copy_elem(dst, flat_of(rank, out_shape, o), src, flat_of(rank, in_shape, j), es);
    } while (next_index(1, rank, out_shape, o));
  }
  return 0;
}

/* One load/store pair in the paper's form (Section 2, equations (load),
 * (store); Section 2.1's pair pattern): for every i in the box
 * 0 <= i_j < bounds[j], in lexicographic order,
 *     v = t_l[C_l i + b_l];   t_s[C_s i + b_s] = v.
 * C matrices are row-major (rank x n_loops).  load_tensor_rank == 0 means the
 * statement stores the constant `fill` (low es bytes).  With guarded != 0 a
 * load whose index leaves t_l's shape yields `fill` instead.  An unguarded
 * access outside its tensor makes the call fail (-3) before anything is
 * written past a buffer.  Stores that collide are last-writer-wins, which is
 * what sequential execution means. */
int oracle_affine_stmt(const void *tl, int l_rank, const int64_t *l_shape, const int64_t *Cl,
                       const int64_t *bl, void *ts, int s_rank, const int64_t *s_shape, const int64_t *Cs,
                       const int64_t *bs, int n_loops, const int64_t *bounds, int guarded,
                       const unsigned char *fill, int es) {
  if (bad_common(s_rank, s_shape, es) || n_loops < 0 || n_loops > ORACLE_MAX_LOOPS) return -1;
  if (l_rank != 0 && bad_common(l_rank, l_shape, es)) return -1;
  int64_t i[ORACLE_MAX_LOOPS + 1] = {0};
  int64_t total = 1;
  for (int k = 0; k < n_loops; ++k) {
    if (bounds[k] < 0) return -2;
    total *= bounds[k];
  }
  const unsigned char *src = (const unsigned char *)tl;
  unsigned char *dst = (unsigned char *)ts;
  for (int64_t cnt = 0; cnt < total; ++cnt) {
    int64_t sidx[ORACLE_MAX_RANK], lidx[ORACLE_MAX_RANK];
    for (int d = 0; d < s_rank; ++d) {
      int64_t v = bs[d];
      for (int k = 0; k < n_loops; ++k) v += Cs[d * n_loops + k] * i[k];
      if (v < 0 || v >= s_shape[d]) return -3;
      sidx[d] = v;
    }
    int use_fill = (l_rank == 0);
    for (int d = 0; d < l_rank; ++d) {
      int64_t v = bl[d];
      for (int k = 0; k < n_loops; ++k) v += Cl[d * n_loops + k] * i[k];
      if (v < 0 || v >= l_shape[d]) {
        if (!guarded) return -3;
        use_fill = 1;
      }
      lidx[d] = v;
    }
    if (use_fill)
      memcpy(dst + flat_of(s_rank, s_shape, sidx) * es, fill, (size_t)es);
    else
      copy_elem(dst, flat_of(s_rank, s_shape, sidx), src, flat_of(l_rank, l_shape, lidx), es);
    if (n_loops > 0) next_index(0, n_loops, bounds, i);
  }
  return 0;
}
