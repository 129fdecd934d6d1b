// Chain builder: writes the load/store loop nest of each common layout
// operator in the paper's form  t_s[C_s i + b_s] = t_l[C_l i + b_l]
// (Section 2, equations (load)/(store); Section 2.1 lists the operator
// families).  Nothing is composed here.
#include <cstring>
#include <new>
#include <vector>

#include "amap_internal.hpp"

namespace {

struct StmtRec {
  std::vector<int64_t> bounds, lC, lb, sC, sb;
  int32_t load_tensor = AMAP_CONST, store_tensor = 0;
  int32_t load_rank = 0, store_rank = 0;
  int32_t guarded = 0;
  uint64_t fill = 0;
};

}  // namespace

struct amap_builder {
  int32_t elem_size = 0;
  std::vector<std::vector<int64_t>> shapes;
  std::vector<int32_t> inputs;
  std::vector<StmtRec> stmts;
  // the view handed out by amap_builder_chain
  std::vector<amap_tensor> v_tensors;
  std::vector<amap_stmt> v_stmts;
  amap_chain v_chain;

  int32_t add_tensor(const std::vector<int64_t> &shape) {
    shapes.push_back(shape);
    return (int32_t)shapes.size() - 1;
  }
  bool valid(int32_t t) const { return t >= 0 && t < (int32_t)shapes.size(); }
};

static bool good_shape(int32_t rank, const int64_t *shape) {
  if (rank < 1 || rank > AMAP_MAX_RANK || !shape) return false;
  for (int d = 0; d < rank; ++d)
    if (shape[d] < 0) return false;
  return true;
}

static std::vector<int64_t> identity_rows(int rank, int n, int first_loop = 0) {
  std::vector<int64_t> C((size_t)rank * n, 0);
  for (int d = 0; d < rank; ++d) C[(size_t)d * n + first_loop + d] = 1;
  return C;
}

#define GUARD_BUILDER(b, out) \
  if (!(b) || !(out)) return AMAP_EINVAL;

extern "C" int amap_builder_create(int32_t elem_size, amap_builder **out) {
  if (!out) return AMAP_EINVAL;
  if (!(elem_size == 1 || elem_size == 2 || elem_size == 4 || elem_size == 8 || elem_size == 16)) return AMAP_EINVAL;
  amap_builder *b = new (std::nothrow) amap_builder();
  if (!b) return AMAP_ENOMEM;
  b->elem_size = elem_size;
  *out = b;
  return AMAP_OK;
}

extern "C" void amap_builder_destroy(amap_builder *b) { delete b; }

extern "C" int amap_builder_input(amap_builder *b, int32_t rank, const int64_t *shape, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!good_shape(rank, shape)) return AMAP_EINVAL;
  *out = b->add_tensor(std::vector<int64_t>(shape, shape + rank));
  b->inputs.push_back(*out);
  return AMAP_OK;
}

extern "C" int amap_builder_opaque(amap_builder *b, int32_t n_ins, const int32_t *ins, int32_t rank, const int64_t *shape,
                                   int32_t *out) {
  GUARD_BUILDER(b, out);
  if (n_ins < 0 || (n_ins > 0 && !ins) || !good_shape(rank, shape)) return AMAP_EINVAL;
  for (int32_t k = 0; k < n_ins; ++k)
    if (!b->valid(ins[k])) return AMAP_EINVAL;
  // to the host algebra the operator's result is one more external tensor
  *out = b->add_tensor(std::vector<int64_t>(shape, shape + rank));
  b->inputs.push_back(*out);
  return AMAP_OK;
}

extern "C" int amap_builder_tensor(amap_builder *b, int32_t rank, const int64_t *shape, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!good_shape(rank, shape)) return AMAP_EINVAL;
  *out = b->add_tensor(std::vector<int64_t>(shape, shape + rank));
  return AMAP_OK;
}

extern "C" int amap_builder_stmt(amap_builder *b, const amap_stmt *st) {
  if (!b || !st) return AMAP_EINVAL;
  const int n = st->n_loops;
  if (n < 0 || n > AMAP_MAX_LOOPS || (n > 0 && !st->bounds)) return AMAP_EINVAL;
  if (!b->valid(st->store.tensor) || !st->store.b || (n > 0 && !st->store.C)) return AMAP_EINVAL;
  StmtRec r;
  r.bounds.assign(st->bounds, st->bounds + n);
  r.store_tensor = st->store.tensor;
  r.store_rank = st->store.rank;
  if (r.store_rank < 1 || r.store_rank > AMAP_MAX_RANK) return AMAP_EINVAL;
  r.sC.assign(st->store.C, st->store.C + (size_t)r.store_rank * n);
  r.sb.assign(st->store.b, st->store.b + r.store_rank);
  r.load_tensor = st->load.tensor;
  if (r.load_tensor != AMAP_CONST) {
    if (!b->valid(r.load_tensor) || !st->load.b || (n > 0 && !st->load.C)) return AMAP_EINVAL;
    r.load_rank = st->load.rank;
    if (r.load_rank < 1 || r.load_rank > AMAP_MAX_RANK) return AMAP_EINVAL;
    r.lC.assign(st->load.C, st->load.C + (size_t)r.load_rank * n);
    r.lb.assign(st->load.b, st->load.b + r.load_rank);
  }
  r.guarded = st->guarded;
  r.fill = st->fill_bits;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

// reshape: loops are the common refinement of the two shapes, so that both
// the load into the old shape and the store into the new one are affine.
extern "C" int amap_builder_reshape(amap_builder *b, int32_t src, int32_t rank, const int64_t *shape, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || !good_shape(rank, shape)) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  const std::vector<int64_t> ou(shape, shape + rank);
  __int128 ni = 1, no = 1;
  for (int64_t v : in) ni *= v;
  for (int64_t v : ou) no *= v;
  if (ni != no) return AMAP_EINVAL;
  StmtRec r;
  std::vector<int> in_dim, out_dim;  // which dimension each refined loop belongs to
  bool aligned = true;
  if (ni > 0) {
    // unit dimensions need no loop: walk the others with two cursors
    std::vector<int> idim, odim;
    for (size_t d = 0; d < in.size(); ++d)
      if (in[d] != 1) idim.push_back((int)d);
    for (size_t d = 0; d < ou.size(); ++d)
      if (ou[d] != 1) odim.push_back((int)d);
    size_t i = 0, j = 0;
    int64_t a = idim.empty() ? 1 : in[idim[0]], c = odim.empty() ? 1 : ou[odim[0]];
    while (i < idim.size() && j < odim.size()) {
      int64_t f;
      if (a == c) f = a;
      else if (a > c && a % c == 0) f = c;
      else if (c > a && c % a == 0) f = a;
      else { aligned = false; break; }  // factors do not line up
      if (r.bounds.size() >= AMAP_MAX_LOOPS) { aligned = false; break; }
      r.bounds.push_back(f);
      in_dim.push_back(idim[i]);
      out_dim.push_back(odim[j]);
      a /= f;
      c /= f;
      if (a == 1 && ++i < idim.size()) a = in[idim[i]];
      if (c == 1 && ++j < odim.size()) c = ou[odim[j]];
    }
  } else {
    r.bounds.push_back(0);
    in_dim.push_back(0);
    out_dim.push_back(0);
  }
  if (!aligned) {
    // No common refinement of the two shapes: one loop over the flat views of both tensors (still an affine pair).
    if (ni > INT64_MAX / 2) return AMAP_EOVERFLOW;
    r.bounds = {(int64_t)ni};
    r.lC = {1};
    r.sC = {1};
    r.lb = {0};
    r.sb = {0};
    r.load_tensor = src;
    r.load_rank = r.store_rank = 1;
    r.store_tensor = b->add_tensor(ou);
    *out = r.store_tensor;
    b->stmts.push_back(std::move(r));
    return AMAP_OK;
  }
  const int n = (int)r.bounds.size();
  auto rows = [&](const std::vector<int64_t> &shp, const std::vector<int> &dim_of) {
    std::vector<int64_t> C(shp.size() * (size_t)n, 0);
    for (size_t d = 0; d < shp.size(); ++d) {
      int64_t mult = 1;
      for (int k = n - 1; k >= 0; --k)
        if (dim_of[k] == (int)d) {
          C[d * n + k] = mult;
          mult *= r.bounds[k];
        }
    }
    return C;
  };
  r.lC = rows(in, in_dim);
  r.sC = rows(ou, out_dim);
  r.lb.assign(in.size(), 0);
  r.sb.assign(ou.size(), 0);
  r.load_tensor = src;
  r.load_rank = (int32_t)in.size();
  r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_transpose(amap_builder *b, int32_t src, int32_t rank, const int32_t *perm, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || !perm || rank != (int32_t)b->shapes[src].size()) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  std::vector<int64_t> ou(rank);
  std::vector<char> seen(rank, 0);
  for (int d = 0; d < rank; ++d) {
    if (perm[d] < 0 || perm[d] >= rank || seen[perm[d]]) return AMAP_EINVAL;
    seen[perm[d]] = 1;
    ou[d] = in[perm[d]];
  }
  StmtRec r;
  r.bounds = ou;  // loops = output index
  r.sC = identity_rows(rank, rank);
  r.sb.assign(rank, 0);
  r.lC.assign((size_t)rank * rank, 0);
  for (int d = 0; d < rank; ++d) r.lC[(size_t)perm[d] * rank + d] = 1;  // in[perm[d]] = o[d]
  r.lb.assign(rank, 0);
  r.load_tensor = src;
  r.load_rank = r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_slice(amap_builder *b, int32_t src, int32_t rank, const int64_t *start, const int64_t *stop,
                                  const int64_t *step, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || !start || !stop || !step || rank != (int32_t)b->shapes[src].size()) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  std::vector<int64_t> ou(rank);
  for (int d = 0; d < rank; ++d) {
    if (step[d] < 1 || start[d] < 0 || stop[d] > in[d] || stop[d] < start[d]) return AMAP_EINVAL;
    ou[d] = (stop[d] - start[d] + step[d] - 1) / step[d];
  }
  StmtRec r;
  r.bounds = ou;
  r.sC = identity_rows(rank, rank);
  r.sb.assign(rank, 0);
  r.lC.assign((size_t)rank * rank, 0);
  for (int d = 0; d < rank; ++d) r.lC[(size_t)d * rank + d] = step[d];
  r.lb.assign(start, start + rank);
  r.load_tensor = src;
  r.load_rank = r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_concat(amap_builder *b, int32_t n, const int32_t *srcs, int32_t axis, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (n < 1 || !srcs || !b->valid(srcs[0])) return AMAP_EINVAL;
  const int rank = (int)b->shapes[srcs[0]].size();
  if (axis < 0 || axis >= rank) return AMAP_EINVAL;
  std::vector<int64_t> ou = b->shapes[srcs[0]];
  ou[axis] = 0;
  for (int q = 0; q < n; ++q) {
    if (!b->valid(srcs[q]) || (int)b->shapes[srcs[q]].size() != rank) return AMAP_EINVAL;
    for (int d = 0; d < rank; ++d)
      if (d != axis && b->shapes[srcs[q]][d] != ou[d]) return AMAP_EINVAL;
    ou[axis] += b->shapes[srcs[q]][axis];
  }
  const int32_t t = b->add_tensor(ou);
  int64_t off = 0;
  for (int q = 0; q < n; ++q) {  // one statement per joined tensor, loops = its own index
    StmtRec r;
    r.bounds = b->shapes[srcs[q]];
    r.lC = identity_rows(rank, rank);
    r.lb.assign(rank, 0);
    r.sC = identity_rows(rank, rank);
    r.sb.assign(rank, 0);
    r.sb[axis] = off;
    off += r.bounds[axis];
    r.load_tensor = srcs[q];
    r.load_rank = r.store_rank = rank;
    r.store_tensor = t;
    b->stmts.push_back(std::move(r));
  }
  *out = t;
  return AMAP_OK;
}

extern "C" int amap_builder_pad(amap_builder *b, int32_t src, int32_t rank, const int64_t *lo, const int64_t *hi,
                                uint64_t fill_bits, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || !lo || !hi || rank != (int32_t)b->shapes[src].size()) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  std::vector<int64_t> ou(rank);
  for (int d = 0; d < rank; ++d) {
    if (lo[d] < 0 || hi[d] < 0) return AMAP_EINVAL;
    ou[d] = lo[d] + in[d] + hi[d];
  }
  StmtRec r;  // loops = output index; the load is guarded: outside the input it yields the fill value
  r.bounds = ou;
  r.sC = identity_rows(rank, rank);
  r.sb.assign(rank, 0);
  r.lC = identity_rows(rank, rank);
  r.lb.resize(rank);
  for (int d = 0; d < rank; ++d) r.lb[d] = -lo[d];
  r.guarded = 1;
  r.fill = fill_bits;
  r.load_tensor = src;
  r.load_rank = r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_window_ex(amap_builder *b, int32_t src, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                                      int32_t dilation, int32_t column_order, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || b->shapes[src].size() != 4 || kh < 1 || kw < 1 || stride < 1 || pad < 0 || dilation < 1 ||
      (column_order != AMAP_WINDOW_COLS_RSC && column_order != AMAP_WINDOW_COLS_CRS))
    return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  const int64_t N = in[0], H = in[1], W = in[2], C = in[3];
  const int64_t span_h = (int64_t)dilation * (kh - 1) + 1, span_w = (int64_t)dilation * (kw - 1) + 1;
  if (H + 2 * pad < span_h || W + 2 * pad < span_w) return AMAP_EINVAL;
  const int64_t Ho = (H + 2 * pad - span_h) / stride + 1, Wo = (W + 2 * pad - span_w) / stride + 1;
  StmtRec r;  // loops (n, ho, wo, r, s, c)
  r.bounds = {N, Ho, Wo, kh, kw, C};
  const int n = 6;
  r.lC.assign(4 * n, 0);
  r.lC[0 * n + 0] = 1;
  r.lC[1 * n + 1] = stride;
  r.lC[1 * n + 3] = dilation;
  r.lC[2 * n + 2] = stride;
  r.lC[2 * n + 4] = dilation;
  r.lC[3 * n + 5] = 1;
  r.lb = {0, -(int64_t)pad, -(int64_t)pad, 0};
  r.sC.assign(2 * n, 0);
  r.sC[0 * n + 0] = Ho * Wo;
  r.sC[0 * n + 1] = Wo;
  r.sC[0 * n + 2] = 1;
  if (column_order == AMAP_WINDOW_COLS_RSC) {  // column (r*kw + s)*C + c
    r.sC[1 * n + 3] = (int64_t)kw * C;
    r.sC[1 * n + 4] = C;
    r.sC[1 * n + 5] = 1;
  } else {  // column (c*kh + r)*kw + s
    r.sC[1 * n + 3] = kw;
    r.sC[1 * n + 4] = 1;
    r.sC[1 * n + 5] = (int64_t)kh * kw;
  }
  r.sb = {0, 0};
  r.guarded = 1;
  r.fill = 0;
  r.load_tensor = src;
  r.load_rank = 4;
  r.store_rank = 2;
  r.store_tensor = b->add_tensor({N * Ho * Wo, (int64_t)kh * kw * C});
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_window(amap_builder *b, int32_t src, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                                   int32_t *out) {
  return amap_builder_window_ex(b, src, kh, kw, stride, pad, 1, AMAP_WINDOW_COLS_RSC, out);
}

extern "C" int amap_builder_tile(amap_builder *b, int32_t src, int32_t rank, const int64_t *reps, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || !reps || rank != (int32_t)b->shapes[src].size() || 2 * rank > AMAP_MAX_LOOPS) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  std::vector<int64_t> ou(rank);
  StmtRec r;  // loops (rep_0, i_0, rep_1, i_1, ...): a load that ignores the rep loops
  const int n = 2 * rank;
  r.lC.assign((size_t)rank * n, 0);
  r.sC.assign((size_t)rank * n, 0);
  for (int d = 0; d < rank; ++d) {
    if (reps[d] < 1) return AMAP_EINVAL;
    ou[d] = reps[d] * in[d];
    r.bounds.push_back(reps[d]);
    r.bounds.push_back(in[d]);
    r.lC[(size_t)d * n + 2 * d + 1] = 1;
    r.sC[(size_t)d * n + 2 * d] = in[d];
    r.sC[(size_t)d * n + 2 * d + 1] = 1;
  }
  r.lb.assign(rank, 0);
  r.sb.assign(rank, 0);
  r.load_tensor = src;
  r.load_rank = r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_repeat(amap_builder *b, int32_t src, int32_t axis, int64_t count, int32_t *out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(src) || count < 1) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  const int rank = (int)in.size();
  if (axis < 0 || axis >= rank || rank + 1 > AMAP_MAX_LOOPS) return AMAP_EINVAL;
  std::vector<int64_t> ou = in;
  ou[axis] = count * in[axis];
  StmtRec r;  // loops (i_0, ..., i_axis, j, ..., i_{rank-1}): the load ignores the copy loop j
  const int n = rank + 1;
  r.lC.assign((size_t)rank * n, 0);
  r.sC.assign((size_t)rank * n, 0);
  for (int d = 0; d < rank; ++d) {
    const int k = d <= axis ? d : d + 1;  // loop of i_d
    r.lC[(size_t)d * n + k] = 1;
    r.sC[(size_t)d * n + k] = d == axis ? count : 1;
  }
  r.sC[(size_t)axis * n + axis + 1] = 1;
  for (int k = 0; k < n; ++k) r.bounds.push_back(k == axis + 1 ? count : in[k <= axis ? k : k - 1]);
  r.lb.assign(rank, 0);
  r.sb.assign(rank, 0);
  r.load_tensor = src;
  r.load_rank = r.store_rank = rank;
  r.store_tensor = b->add_tensor(ou);
  *out = r.store_tensor;
  b->stmts.push_back(std::move(r));
  return AMAP_OK;
}

extern "C" int amap_builder_split(amap_builder *b, int32_t src, int32_t axis, int32_t n_parts, const int64_t *sizes,
                                  int32_t *outs) {
  GUARD_BUILDER(b, outs);
  if (!b->valid(src) || !sizes || n_parts < 1) return AMAP_EINVAL;
  const std::vector<int64_t> in = b->shapes[src];
  const int rank = (int)in.size();
  if (axis < 0 || axis >= rank) return AMAP_EINVAL;
  int64_t total = 0;
  for (int q = 0; q < n_parts; ++q) {
    if (sizes[q] < 0) return AMAP_EINVAL;
    total += sizes[q];
  }
  if (total != in[axis]) return AMAP_EINVAL;
  int64_t off = 0;
  for (int q = 0; q < n_parts; ++q) {  // one statement and one tensor per part, loops = the part's own index
    StmtRec r;
    r.bounds = in;
    r.bounds[axis] = sizes[q];
    r.lC = identity_rows(rank, rank);
    r.lb.assign(rank, 0);
    r.lb[axis] = off;
    off += sizes[q];
    r.sC = identity_rows(rank, rank);
    r.sb.assign(rank, 0);
    r.load_tensor = src;
    r.load_rank = r.store_rank = rank;
    r.store_tensor = b->add_tensor(r.bounds);
    outs[q] = r.store_tensor;
    b->stmts.push_back(std::move(r));
  }
  return AMAP_OK;
}

extern "C" int amap_builder_chain(amap_builder *b, int32_t output, const amap_chain **out) {
  GUARD_BUILDER(b, out);
  if (!b->valid(output)) return AMAP_EINVAL;
  b->v_tensors.clear();
  for (auto &s : b->shapes) b->v_tensors.push_back({(int32_t)s.size(), s.data()});
  b->v_stmts.clear();
  for (auto &r : b->stmts) {
    amap_stmt st;
    memset(&st, 0, sizeof st);
    st.n_loops = (int32_t)r.bounds.size();
    st.bounds = r.bounds.data();
    st.load = {r.load_tensor, r.load_rank, r.lC.data(), r.lb.data()};
    st.store = {r.store_tensor, r.store_rank, r.sC.data(), r.sb.data()};
    st.guarded = r.guarded;
    st.fill_bits = r.fill;
    b->v_stmts.push_back(st);
  }
  b->v_chain.n_tensors = (int32_t)b->v_tensors.size();
  b->v_chain.tensors = b->v_tensors.data();
  b->v_chain.n_stmts = (int32_t)b->v_stmts.size();
  b->v_chain.stmts = b->v_stmts.data();
  b->v_chain.n_inputs = (int32_t)b->inputs.size();
  b->v_chain.inputs = b->inputs.data();
  b->v_chain.output = output;
  b->v_chain.elem_size = b->elem_size;
  *out = &b->v_chain;
  return AMAP_OK;
}
