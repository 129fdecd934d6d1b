// amap_compose: data-movement elimination on the host (the paper's Section
// 2.1).  For a pair  v = t_l[f_l(i)],  t_s[f_s(i)] = v  and a reader
// v' = t_s[f_l'(i')]  the paper forms the reverse f_s' of the store map,
// g_ls = f_l o f_s' (equation (1)) and g' = g_ls o f_l' (equation (2)), rewrites
// the reader to load t_l[g'(i')] and drops t_s; this is repeated until no
// intermediate tensor is left.
//
// Design here: tensors are dense and row-major, so every access is first
// linearised to a flat element offset  b + sum_k stride_k i_k.  The reverse of
// a store is in general only quasi-affine (floor-div / mod), so it is never
// written down as a function of the tensor index.  Instead the READER's loop
// nest is kept as the domain and refined: the store's loops, sorted by stride,
// are the digits of a mixed-radix number system over t_s's flat offsets, and a
// reader loop is assigned to the digit its stride falls on -- and split in two
// when it runs across a digit boundary (that is how reshapes compose).  Each
// digit becomes an affine function delta_k(i') of the reader's loops, i.e.
// f_s'(f_l'(i')) restricted to where every delta_k lies inside its loop's
// bounds; g' follows by substituting delta into f_l.  A tensor defined by
// several statements (concat) or only partly (pad) yields one piece per
// writer.  Soundness does not rest on the matching heuristics: the pieces
// produced for a reader are exact preimages, pairwise disjoint, and their
// point counts must add up to the reader's domain, otherwise the call fails.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>

#include "amap_internal.hpp"
#define AMAP_DEVICE_STRUCTS_ONLY
#include "amap_device.h"

namespace amap {

static Status err(int code, const std::string &m) {
  Status s;
  s.code = code;
  s.msg = m;
  return s;
}

static inline int64_t floordiv(int64_t a, int64_t b) {
  int64_t q = a / b, r = a % b;
  return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q;
}
static inline int64_t ceildiv(int64_t a, int64_t b) { return -floordiv(-a, b); }

static const int64_t kBig = INT64_MAX / 4;
static const int kMaxPieceConstraints = 6;  // = the device descriptor's constraint slots
static const int kMaxPiecesPerReader = 64;  // a reader that shatters into more pieces is cheaper through a temporary

// ---------------------------------------------------------------------------
// linearisation and validation of one access
// ---------------------------------------------------------------------------
struct Rows {
  std::vector<Aff> row;  // one affine expression per tensor dimension
};

static Status read_access(const amap_access &a, int n, const std::vector<TensorInfo> &T, Rows *rows, bool *flat) {
  if (a.tensor < 0 || a.tensor >= (int)T.size()) return err(AMAP_EINVAL, "access names an unknown tensor");
  const TensorInfo &t = T[a.tensor];
  // an access of rank 1 to a tensor of higher rank addresses its flat row-major view
  *flat = (a.rank == 1 && t.shape.size() > 1);
  if (!*flat && a.rank != (int)t.shape.size()) return err(AMAP_EINVAL, "access rank differs from the tensor's rank");
  if (!a.b || (n > 0 && !a.C)) return err(AMAP_EINVAL, "null C or b");
  rows->row.resize(a.rank);
  for (int d = 0; d < a.rank; ++d) {
    rows->row[d].c0 = a.b[d];
    rows->row[d].c.assign(a.C ? a.C + (size_t)d * n : nullptr, a.C ? a.C + (size_t)(d + 1) * n : nullptr);
    rows->row[d].c.resize(n, 0);
  }
  return Status();
}

static bool linearise(const Rows &r, const TensorInfo &t, int n, Aff *out) {
  __int128 c0 = 0;
  std::vector<__int128> c(n, 0);
  for (size_t d = 0; d < r.row.size(); ++d) {
    c0 += (__int128)r.row[d].c0 * t.stride[d];
    for (int k = 0; k < n; ++k) c[k] += (__int128)r.row[d].c[k] * t.stride[d];
  }
  out->c.resize(n);
  if (c0 > kBig || c0 < -kBig) return false;
  out->c0 = (int64_t)c0;
  for (int k = 0; k < n; ++k) {
    if (c[k] > kBig || c[k] < -kBig) return false;
    out->c[k] = (int64_t)c[k];
  }
  return true;
}

// ---------------------------------------------------------------------------
// store checks
// ---------------------------------------------------------------------------
static void enumerate_offsets(const Piece &p, std::vector<int64_t> *out) {
  int64_t total = 1;
  for (int64_t e : p.ext) total *= e;
  out->reserve(out->size() + total);
  std::vector<int64_t> idx(p.ext.size(), 0);
  for (int64_t t = 0; t < total; ++t) {
    int64_t v = p.dst.c0;
    for (size_t k = 0; k < idx.size(); ++k) v += p.dst.c[k] * idx[k];
    out->push_back(v);
    for (int k = (int)idx.size() - 1; k >= 0; --k) {
      if (++idx[k] < p.ext[k]) break;
      idx[k] = 0;
    }
  }
}

static int64_t box_points(const Piece &p) {
  __int128 t = 1;
  for (int64_t e : p.ext) {
    t *= e;
    if (t > kBig) return -1;
  }
  return (int64_t)t;
}

// strides sorted descending, each larger than everything the lower loops can add up to
static bool nested_strides(const std::vector<int64_t> &d, const std::vector<int64_t> &e) {
  __int128 below = 0;
  for (int k = (int)d.size() - 1; k >= 0; --k) {
    if (d[k] <= below) return false;
    below += (__int128)d[k] * (e[k] - 1);
  }
  return true;
}

static Status check_injective(const Piece &raw) {
  Piece p = raw;
  p.guards.clear();
  p.domain.clear();
  drop_unit_loops(p);
  for (int k = 0; k < p.n(); ++k) {
    if (p.dst.c[k] == 0) return err(AMAP_ESTORE_NOT_INJECTIVE, "a loop does not move the store");
    if (p.dst.c[k] < 0) reverse_loop(p, k);
  }
  std::vector<int> order(p.n());
  std::iota(order.begin(), order.end(), 0);
  std::sort(order.begin(), order.end(), [&](int a, int b) { return p.dst.c[a] > p.dst.c[b]; });
  permute_loops(p, order);
  if (nested_strides(p.dst.c, p.ext)) return Status();
  const int64_t pts = box_points(p);
  if (pts < 0 || pts > (1 << 22)) return err(AMAP_EUNSUPPORTED, "cannot decide whether a large interleaved store is injective");
  std::vector<int64_t> offs;
  enumerate_offsets(p, &offs);
  std::sort(offs.begin(), offs.end());
  if (std::adjacent_find(offs.begin(), offs.end()) != offs.end())
    return err(AMAP_ESTORE_NOT_INJECTIVE, "two loop points store to the same element");
  return Status();
}

struct RawStore {
  Piece piece;                    // dst only
  std::vector<int64_t> lo, hi;    // per tensor dimension index range
  std::vector<int64_t> step, rem; // per dimension: index = rem (mod step) when a single loop drives it, else step 1
};

struct TensorState {
  std::vector<RawStore> stores;
  std::vector<bool> bitmap;  // built lazily when interval tests are inconclusive
  bool has_bitmap = false;
  std::vector<Piece> defs;  // composed definitions (sources are external tensor ids or AMAP_CONST)
  int64_t defined_points = 0;
};

static bool surely_disjoint(const RawStore &a, const RawStore &b) {
  if (a.lo.size() != b.lo.size()) return false;  // one of them addresses the flat view
  for (size_t d = 0; d < a.lo.size(); ++d) {
    if (a.hi[d] < b.lo[d] || b.hi[d] < a.lo[d]) return true;
    const int64_t g = std::gcd(a.step[d], b.step[d]);
    if (g > 1 && ((a.rem[d] - b.rem[d]) % g) != 0) return true;
  }
  return false;
}

static Status mark_bitmap(TensorState &ts, const Piece &p) {
  std::vector<int64_t> offs;
  enumerate_offsets(p, &offs);
  for (int64_t o : offs) {
    if (ts.bitmap[o]) return err(AMAP_EOVERLAP, "two statements store to the same element");
    ts.bitmap[o] = true;
  }
  return Status();
}

static Status check_overlap(TensorState &ts, const TensorInfo &ti, const RawStore &neu) {
  bool need_exact = ts.has_bitmap;
  if (!need_exact)
    for (auto &old : ts.stores)
      if (!surely_disjoint(old, neu)) {
        need_exact = true;
        break;
      }
  if (!need_exact) return Status();
  if (!ts.has_bitmap) {
    int64_t pts = box_points(neu.piece);
    for (auto &old : ts.stores) pts += box_points(old.piece);
    if (ti.numel > (1ll << 28) || pts > (1ll << 28))
      return err(AMAP_EUNSUPPORTED, "cannot prove that two large statements write disjoint elements");
    ts.bitmap.assign(ti.numel, false);
    ts.has_bitmap = true;
    for (auto &old : ts.stores) {
      Status s = mark_bitmap(ts, old.piece);
      if (!s.ok()) return s;
    }
  }
  return mark_bitmap(ts, neu.piece);
}

// ---------------------------------------------------------------------------
// composing one reader with one writer piece
// ---------------------------------------------------------------------------
struct PairResult {
  Piece q;                  // ext, dst, src, srcoff, fill (of the writer); no constraints yet
  std::vector<Con> dR, gR;  // the reader's own domain / guards, refined
  std::vector<Con> dNew;    // digit ranges and the writer's domain, in the reader's loops
  std::vector<Con> gW;      // the writer's guards, in the reader's loops
};

static void split_loop(Piece &p, int j, int64_t f) {
  // i_j = f * q + t, q < ext/f (position j), t < f (position j+1)
  auto sp = [&](Aff &a) {
    const int64_t c = a.c[j];
    a.c[j] = c * f;
    a.c.insert(a.c.begin() + j + 1, c);
  };
  sp(p.dst);
  if (p.src != AMAP_CONST) sp(p.srcoff);
  if (p.src != AMAP_CONST && p.qa.on) sp(p.qa.f);
  for (auto &g : p.guards) sp(g.e);
  for (auto &g : p.domain) sp(g.e);
  const int64_t e = p.ext[j];
  p.ext[j] = e / f;
  p.ext.insert(p.ext.begin() + j + 1, f);
}

static Aff substitute(const Aff &a, const std::vector<Aff> &delta, const std::vector<int> &digit_of_loop, int n_reader) {
  Aff r;
  r.c0 = a.c0;
  r.c.assign(n_reader, 0);
  for (size_t k = 0; k < a.c.size(); ++k) {
    if (a.c[k] == 0) continue;
    const Aff &d = delta[digit_of_loop[k]];
    r.c0 += a.c[k] * d.c0;
    for (int j = 0; j < n_reader; ++j) r.c[j] += a.c[k] * d.c[j];
  }
  return r;
}

static Status compose_pair(const Piece &R, const Piece &W, std::vector<PairResult> *out) {
  // canonical writer: unit loops gone, positive strides, sorted descending
  Piece Wc = W;
  drop_unit_loops(Wc);
  for (int k = 0; k < Wc.n(); ++k) {
    if (Wc.dst.c[k] == 0) return err(AMAP_ESTORE_NOT_INJECTIVE, "a loop does not move the store");
    if (Wc.dst.c[k] < 0) reverse_loop(Wc, k);
  }
  {
    std::vector<int> order(Wc.n());
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int a, int b) { return Wc.dst.c[a] > Wc.dst.c[b]; });
    permute_loops(Wc, order);
  }
  if (!nested_strides(Wc.dst.c, Wc.ext))
    return err(AMAP_EUNSUPPORTED, "the store of a tensor that is read again interleaves its loops");
  // digits of the writer's number system; a trailing unit digit absorbs what no loop reaches
  std::vector<int64_t> dd = Wc.dst.c, de = Wc.ext;
  const int real_digits = (int)dd.size();
  if (dd.empty() || dd.back() > 1) {
    dd.push_back(1);
    de.push_back(1);
  }
  const int K = (int)dd.size();

  Piece Rc = R;
  for (int j = 0; j < Rc.n(); ++j)
    if (Rc.srcoff.c[j] < 0) reverse_loop(Rc, j);

  std::vector<std::vector<int64_t>> M(K);  // M[k][j]: reader loop j adds M[k][j] * i_j to digit k
  for (int j = 0; j < Rc.n();) {
    for (auto &row : M) row.resize(Rc.n(), 0);
    const int64_t r = Rc.srcoff.c[j], E = Rc.ext[j];
    if (r == 0 || E == 1) {
      ++j;
      continue;
    }
    int k = 0;
    while (dd[k] > r) ++k;  // dd[K-1] == 1 <= r
    if (r % dd[k] == 0 && k > 0 && dd[k - 1] % dd[k] == 0) {
      const int64_t m = r / dd[k], cap = dd[k - 1] / dd[k];
      if ((__int128)m * (E - 1) >= cap && cap % m == 0) {
        const int64_t f = cap / m;
        if (f > 1 && E % f == 0) {
          split_loop(Rc, j, f);
          for (auto &row : M) row.insert(row.begin() + j + 1, 0);
          continue;  // look at the outer half again, then the inner one
        }
      }
    }
    int64_t rem = r;
    for (int q = k; q < K; ++q) {
      M[q][j] = rem / dd[q];
      rem -= M[q][j] * dd[q];
    }
    ++j;
  }
  for (auto &row : M) row.resize(Rc.n(), 0);
  const int nR = Rc.n();

  // the constant: every way of spreading it over the digits that leaves each digit a chance to be in range
  std::vector<int64_t> Mx(K, 0);
  for (int k = 0; k < K; ++k)
    for (int j = 0; j < nR; ++j) Mx[k] += M[k][j] * (Rc.ext[j] - 1);
  std::vector<__int128> Lmin(K + 1, 0), Lmax(K + 1, 0);  // what digits > k can add up to
  for (int k = K - 1; k >= 0; --k) {
    Lmin[k] = Lmin[k + 1] - (__int128)dd[k] * Mx[k];
    Lmax[k] = Lmax[k + 1] + (__int128)dd[k] * (de[k] - 1);
  }
  std::vector<std::vector<int64_t>> consts;
  {
    struct Frame {
      int k;
      __int128 rho;
    };
    // depth-first enumeration with an explicit stack
    std::vector<std::pair<Frame, std::vector<int64_t>>> todo;
    todo.push_back({{0, (__int128)Rc.srcoff.c0 - Wc.dst.c0}, std::vector<int64_t>(K, 0)});
    while (!todo.empty()) {
      auto item = todo.back();
      todo.pop_back();
      const int k = item.first.k;
      const __int128 rho = item.first.rho;
      if (k == K) {
        if (rho == 0) consts.push_back(item.second);
        if (consts.size() > 4096) return err(AMAP_EUNSUPPORTED, "too many carry patterns");
        continue;
      }
      // need Lmin[k+1] <= rho - d*c <= Lmax[k+1] and -Mx <= c <= e-1
      __int128 lo128 = rho - Lmax[k + 1], hi128 = rho - Lmin[k + 1];
      // ceil(lo/d), floor(hi/d) with d > 0
      auto fdiv = [](__int128 a, __int128 b) {
        __int128 q = a / b, r = a % b;
        return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q;
      };
      __int128 clo = -fdiv(-lo128, dd[k]), chi = fdiv(hi128, dd[k]);
      clo = std::max<__int128>(clo, -(__int128)Mx[k]);
      chi = std::min<__int128>(chi, de[k] - 1);
      for (__int128 c = clo; c <= chi; ++c) {
        auto nxt = item.second;
        nxt[k] = (int64_t)c;
        todo.push_back({{k + 1, rho - c * dd[k]}, nxt});
      }
    }
  }

  std::vector<int> digit_of_loop(real_digits);
  std::iota(digit_of_loop.begin(), digit_of_loop.end(), 0);
  for (auto &cs : consts) {
    std::vector<Aff> delta(K);
    for (int k = 0; k < K; ++k) {
      delta[k].c0 = cs[k];
      delta[k].c = M[k];
    }
    PairResult pr;
    pr.q.ext = Rc.ext;
    pr.q.dst = Rc.dst;
    pr.q.src = Wc.src;
    pr.q.fill = Wc.fill;
    if (Wc.src != AMAP_CONST)
      pr.q.srcoff = substitute(Wc.srcoff, delta, digit_of_loop, nR);
    else
      pr.q.srcoff.c.assign(nR, 0);
    if (Wc.src != AMAP_CONST && Wc.qa.on) {  // a quasi-affine writer stays one: its inner form follows the reader's loops
      pr.q.qa = Wc.qa;
      pr.q.qa.f = substitute(Wc.qa.f, delta, digit_of_loop, nR);
    }
    pr.dR = Rc.domain;
    pr.gR = Rc.guards;
    for (int k = 0; k < K; ++k) {
      Con c;
      c.e = delta[k];
      c.extent = de[k];
      pr.dNew.push_back(c);
    }
    for (auto &g : Wc.domain) {
      Con c;
      c.e = substitute(g.e, delta, digit_of_loop, nR);
      c.extent = g.extent;
      pr.dNew.push_back(c);
    }
    for (auto &g : Wc.guards) {
      Con c;
      c.e = substitute(g.e, delta, digit_of_loop, nR);
      c.extent = g.extent;
      pr.gW.push_back(c);
    }
    out->push_back(std::move(pr));
  }
  return Status();
}

static void append(std::vector<Con> &a, const std::vector<Con> &b) { a.insert(a.end(), b.begin(), b.end()); }

// Rewrites reader R (whose load names intermediate tensor t) to load external
// tensors directly: equation (2) applied with every statement that defines t.
static Status compose_reader_affine(const Piece &R, const TensorState &ts, const TensorInfo &ti, std::vector<Piece> *out) {
  Piece Rin = R;  // the part of the reader that really loads
  append(Rin.domain, Rin.guards);
  Rin.guards.clear();
  const int64_t need = count_points(Rin);
  if (need < 0) return err(AMAP_EUNSUPPORTED, "cannot count the points of a guarded reader");

  struct Cand {
    PairResult pr;
    Piece in;
  };
  std::vector<Cand> cands;
  int64_t have = 0;
  if (need > 0)
    for (const Piece &W : ts.defs) {
      std::vector<PairResult> prs;
      Status s = compose_pair(R, W, &prs);
      if (!s.ok()) return s;
      for (auto &pr : prs) {
        Piece in = pr.q;
        in.domain = pr.dR;
        append(in.domain, pr.gR);
        append(in.domain, pr.dNew);
        in.guards = pr.gW;
        if (!tighten(in)) continue;
        const int64_t c = count_points(in);
        if (c < 0) return err(AMAP_EUNSUPPORTED, "cannot count the points of a composed piece");
        if (c == 0) continue;
        have += c;
        cands.push_back({std::move(pr), std::move(in)});
      }
    }
  // the kernels evaluate at most kMaxPieceConstraints constraints per piece: beyond that the pair is not worth
  // eliminating (the caller keeps the tensor as a temporary instead)
  for (auto &c : cands)
    if (c.in.guards.size() + c.in.domain.size() + R.guards.size() > (size_t)kMaxPieceConstraints)
      return err(AMAP_EUNSUPPORTED, "the composed piece needs too many constraints");
  if (cands.size() > (size_t)kMaxPiecesPerReader) return err(AMAP_EUNSUPPORTED, "the pair shatters into too many pieces");
  if (have != need) {
    if (ts.defined_points < ti.numel && have < need)
      return err(AMAP_EUNDEFINED, "a statement reads elements of an intermediate tensor that nothing writes");
    return err(AMAP_EUNSUPPORTED, "the reader's loops do not line up with the loops that wrote the tensor");
  }
  if (R.guards.empty()) {
    for (auto &c : cands) out->push_back(std::move(c.in));
    return Status();
  }
  // One writer covers everything the guarded reader loads: keep ONE piece whose
  // guards are the reader's (plus the writer's), instead of a copy piece and
  // separate fill pieces with multi-loop domains.
  if (cands.size() == 1) {
    const PairResult &pr = cands[0].pr;
    const bool w_fill = (pr.q.src == AMAP_CONST);
    if ((pr.gW.empty() && !w_fill) || pr.q.fill == R.fill) {
      Piece f = pr.q;
      f.fill = R.fill;
      f.domain = pr.dR;
      if (!w_fill) {
        f.guards = pr.gR;
        append(f.guards, pr.gW);
      }
      if (tighten(f)) out->push_back(std::move(f));
      return Status();
    }
  }
  for (auto &c : cands) out->push_back(std::move(c.in));
  // where a guard fails: fill pieces, made disjoint by requiring the earlier guards to hold
  for (size_t m = 0; m < R.guards.size(); ++m) {
    for (int side = 0; side < 2; ++side) {
      Piece f;
      f.ext = R.ext;
      f.dst = R.dst;
      f.src = AMAP_CONST;
      f.srcoff.c.assign(R.ext.size(), 0);
      f.fill = R.fill;
      f.domain = R.domain;
      for (size_t q = 0; q < m; ++q) f.domain.push_back(R.guards[q]);
      Con c;
      c.e = R.guards[m].e;
      c.extent = kBig;
      if (side == 0) {  // e < 0  <=>  0 <= -e-1
        c.e.c0 = -c.e.c0 - 1;
        for (auto &v : c.e.c) v = -v;
      } else {  // e >= extent
        c.e.c0 -= R.guards[m].extent;
      }
      f.domain.push_back(c);
      if (tighten(f)) out->push_back(std::move(f));
    }
  }
  return Status();
}

// Where equation (2) has no affine form (a reshape whose factors do not line up with the loops around it), the
// composition still exists as a QUASI-affine map: the reader's offset f(i') into t_s is split into the digits of the
// writer's loop nest (floor-division and remainder by compile-time constants), and those digits go through the
// writer's load.  Supported when one statement wrote t_s, unguarded, as a dense renumbering of all of it.  Such a
// piece pays divisions per access, so it is only worth having where whole runs share them (a contiguous run of at
// least 16 bytes on both sides); otherwise the caller keeps t_s as a temporary -- unless `force`.
static const int kMaxQuasiDigits = 6;
static const int kQuasiPreferredOverPieces = 8;

static Status compose_reader_quasi(const Piece &R, const TensorState &ts, const TensorInfo &ti, int es, bool force,
                                   std::vector<Piece> *out) {
  if (ts.defs.size() != 1) return err(AMAP_EUNSUPPORTED, "quasi-affine composition needs a single writer");
  const Piece &W = ts.defs[0];
  if (W.src == AMAP_CONST || W.qa.on || !W.guards.empty() || !W.domain.empty())
    return err(AMAP_EUNSUPPORTED, "quasi-affine composition needs a plain writer");
  if (ti.numel >= (1ll << 31)) return err(AMAP_EUNSUPPORTED, "tensor too large for a quasi-affine piece");
  Piece Wc = W;
  drop_unit_loops(Wc);
  for (int k = 0; k < Wc.n(); ++k) {
    if (Wc.dst.c[k] == 0) return err(AMAP_ESTORE_NOT_INJECTIVE, "a loop does not move the store");
    if (Wc.dst.c[k] < 0) reverse_loop(Wc, k);
  }
  std::vector<int> order(Wc.n());
  std::iota(order.begin(), order.end(), 0);
  std::sort(order.begin(), order.end(), [&](int a, int b) { return Wc.dst.c[a] > Wc.dst.c[b]; });
  permute_loops(Wc, order);
  // dense: the writer's loops are exactly the digits of t_s's flat offsets
  int64_t place = 1;
  for (int k = Wc.n() - 1; k >= 0; --k) {
    if (Wc.dst.c[k] != place) return err(AMAP_EUNSUPPORTED, "the writer does not number the tensor densely");
    place *= Wc.ext[k];
  }
  if (Wc.dst.c0 != 0 || place != ti.numel || Wc.n() < 1 || Wc.n() > kMaxQuasiDigits)
    return err(AMAP_EUNSUPPORTED, "the writer does not number the tensor densely");
  if (R.guards.size() + R.domain.size() > (size_t)kMaxPieceConstraints)
    return err(AMAP_EUNSUPPORTED, "the composed piece needs too many constraints");
  Piece Q;
  Q.ext = R.ext;
  Q.dst = R.dst;
  Q.src = Wc.src;
  Q.fill = R.fill;
  Q.guards = R.guards;
  Q.domain = R.domain;
  Q.srcoff.c0 = Wc.srcoff.c0;
  Q.srcoff.c.assign(R.ext.size(), 0);
  Q.qa.on = true;
  Q.qa.f = R.srcoff;
  Q.qa.radix = Wc.ext;
  Q.qa.stride = Wc.srcoff.c;
  if (!force) {
    bool worth = false;
    for (int k = 0; k < Q.n() && !worth; ++k) worth = piece_run_elems(Q, k, 64) * es >= 16;
    if (!worth) return err(AMAP_EUNSUPPORTED, "a quasi-affine piece without runs is slower than a temporary");
  }
  if (tighten(Q)) out->push_back(std::move(Q));
  return Status();
}

// quasi: 0 = where no affine composition exists and runs survive, 1 = wherever the pair allows one (also in place
// of an affine composition), -1 = never
static Status compose_reader(const Piece &R, const TensorState &ts, const TensorInfo &ti, int es, int quasi,
                             std::vector<Piece> *out) {
  const size_t before = out->size();
  if (quasi > 0) {
    if (compose_reader_quasi(R, ts, ti, es, true, out).ok()) return Status();
    out->resize(before);
  }
  Status s = compose_reader_affine(R, ts, ti, out);
  if (quasi != 0) return s;
  // no affine composition, or one that shatters the reader into many pieces (one descriptor and one set of
  // constraints each; measured: 64 pieces of 16 KiB runs ran at a fortieth of the one quasi-affine piece's rate)
  const bool shattered = s.ok() && out->size() - before > (size_t)kQuasiPreferredOverPieces;
  if (s.code != AMAP_EUNSUPPORTED && !shattered) return s;
  std::vector<Piece> affine(out->begin() + before, out->end());
  out->resize(before);
  if (compose_reader_quasi(R, ts, ti, es, false, out).ok()) return Status();
  out->resize(before);
  out->insert(out->end(), affine.begin(), affine.end());
  return s;
}

// ---------------------------------------------------------------------------
static int64_t unique_reads(const Piece &p0, int64_t in_numel) {
  Piece p = p0;
  const int64_t pts = count_points(p);
  if (p.src == AMAP_CONST) return 0;
  if (p.qa.on) return std::min(pts >= 0 ? pts : in_numel, in_numel);
  drop_unit_loops(p);
  std::vector<std::pair<int64_t, int64_t>> se;
  for (int k = 0; k < p.n(); ++k)
    if (p.srcoff.c[k] != 0) se.push_back({std::llabs(p.srcoff.c[k]), p.ext[k]});
  std::sort(se.begin(), se.end(), [](auto &a, auto &b) { return a.first > b.first; });
  std::vector<int64_t> d, e;
  for (auto &x : se) {
    d.push_back(x.first);
    e.push_back(x.second);
  }
  int64_t distinct = 1;
  for (int64_t v : e) distinct *= v;
  int64_t bound = (pts >= 0) ? pts : distinct;
  if (nested_strides(d, e)) bound = std::min(bound, distinct);
  return std::min(bound, in_numel);
}

// `outputs`: the tensors wanted as results (one: the chain's own output).  Each becomes a set of pieces of the
// final stage; a tensor may be both an output and read by later statements.
static Status compose_chain(const amap_chain *ch, const std::vector<int> &outputs, uint32_t flags, Map *out) {
  if (!ch) return err(AMAP_EINVAL, "null chain");
  const int es = ch->elem_size;
  if (!(es == 1 || es == 2 || es == 4 || es == 8 || es == 16)) return err(AMAP_EINVAL, "elem_size must be 1, 2, 4, 8 or 16");
  if (ch->n_tensors < 1 || !ch->tensors || ch->n_stmts < 0 || (ch->n_stmts > 0 && !ch->stmts) || ch->n_inputs < 0 ||
      (ch->n_inputs > 0 && !ch->inputs))
    return err(AMAP_EINVAL, "bad chain header");
  if (outputs.empty() || outputs.size() > 8) return err(AMAP_EINVAL, "a map has 1 to 8 outputs");
  for (size_t k = 0; k < outputs.size(); ++k) {
    if (outputs[k] < 0 || outputs[k] >= ch->n_tensors) return err(AMAP_EINVAL, "bad output tensor id");
    for (size_t j = 0; j < k; ++j)
      if (outputs[j] == outputs[k]) return err(AMAP_EINVAL, "an output tensor is named twice");
  }

  std::vector<TensorInfo> T(ch->n_tensors);
  for (int t = 0; t < ch->n_tensors; ++t) {
    const amap_tensor &a = ch->tensors[t];
    if (a.rank < 1 || a.rank > AMAP_MAX_RANK || !a.shape) return err(AMAP_EINVAL, "tensor rank out of range");
    T[t].shape.assign(a.shape, a.shape + a.rank);
    T[t].stride.assign(a.rank, 1);
    __int128 n = 1;
    for (int d = a.rank - 1; d >= 0; --d) {
      if (a.shape[d] < 0) return err(AMAP_EINVAL, "negative extent");
      T[t].stride[d] = (int64_t)n;
      n *= a.shape[d];
      if (n * es > kBig) return err(AMAP_EOVERFLOW, "tensor too large");
    }
    T[t].numel = (int64_t)n;
  }
  for (int q = 0; q < ch->n_inputs; ++q) {
    const int t = ch->inputs[q];
    if (t < 0 || t >= ch->n_tensors || T[t].input_slot >= 0) return err(AMAP_EINVAL, "bad or repeated input tensor id");
    T[t].input_slot = q;
  }
  for (int t : outputs)
    if (T[t].input_slot >= 0) return err(AMAP_EINVAL, "the output tensor is an input");

  std::vector<TensorState> S(ch->n_tensors);
  out->elem_size = es;
  out->in_numel.resize(ch->n_inputs);
  for (int q = 0; q < ch->n_inputs; ++q) out->in_numel[q] = T[ch->inputs[q]].numel;

  // closes the definitions of tensor t: canonical pieces that write temporary `temp`, or (temp < 0) output `out_k`
  auto close_tensor = [&](int t, int temp, int out_k, std::vector<Piece> *done) -> Status {
    std::vector<Piece> pieces = S[t].defs;
    int64_t covered = 0;
    for (auto &p : pieces) {
      const int64_t c = count_points(p);
      if (c < 0) return err(AMAP_EUNSUPPORTED, "cannot count the points of a piece");
      covered += c;
      if (p.src != AMAP_CONST) p.src = T[p.src].input_slot;
    }
    if (covered != T[t].numel)
      return err(temp < 0 ? AMAP_EUNDEFINED : AMAP_EUNSUPPORTED,
                 temp < 0 ? "some output elements are never written" : "a partly written intermediate cannot be kept as a temporary");
    Status s = canonicalise(pieces);
    if (!s.ok()) return s;
    for (auto &p : pieces) {
      p.out = temp < 0 ? out_k : 0;
      for (int k = 0; k < p.n(); ++k)
        if (p.ext[k] > INT32_MAX) return err(AMAP_EOVERFLOW, "a merged loop exceeds 2^31-1 iterations");
    }
    done->insert(done->end(), pieces.begin(), pieces.end());
    return Status();
  };
  auto finish_stage = [&](int t, int temp) -> Status {
    std::vector<Piece> pieces;
    Status s = close_tensor(t, temp, 0, &pieces);
    if (!s.ok()) return s;
    StageInfo st;
    st.first_piece = (int)out->pieces.size();
    st.n_pieces = (int)pieces.size();
    st.dst_temp = temp;
    st.numel = T[t].numel;
    out->stages.push_back(st);
    out->pieces.insert(out->pieces.end(), pieces.begin(), pieces.end());
    return Status();
  };
  auto materialise = [&](int t) -> Status {
    const int k = (int)out->temp_numel.size();
    Status s = finish_stage(t, k);
    if (!s.ok()) return s;
    out->temp_numel.push_back(T[t].numel);
    T[t].input_slot = ch->n_inputs + k;
    S[t].defs.clear();
    return Status();
  };

  for (int si = 0; si < ch->n_stmts; ++si) {
    const amap_stmt &st = ch->stmts[si];
    const int n = st.n_loops;
    if (n < 0 || n > AMAP_MAX_LOOPS || (n > 0 && !st.bounds)) return err(AMAP_EINVAL, "bad loop count");
    bool empty = false;
    for (int k = 0; k < n; ++k) {
      if (st.bounds[k] < 0) return err(AMAP_EINVAL, "negative loop bound");
      if (st.bounds[k] == 0) empty = true;
    }
    if (st.store.tensor == AMAP_CONST) return err(AMAP_EINVAL, "a store needs a tensor");
    Rows srow, lrow;
    bool sflat = false, lflat = false;
    Status s = read_access(st.store, n, T, &srow, &sflat);
    if (!s.ok()) return s;
    const int tsid = st.store.tensor;
    TensorInfo sview = T[tsid], lview;
    if (sflat) {
      sview.shape = {T[tsid].numel};
      sview.stride = {1};
    }
    if (T[tsid].input_slot >= 0)
      return err(AMAP_EINVAL, T[tsid].input_slot < ch->n_inputs ? "a statement stores to an external input"
                                                                : "a statement stores to a tensor after it was read");
    const bool is_const = (st.load.tensor == AMAP_CONST);
    if (!is_const) {
      s = read_access(st.load, n, T, &lrow, &lflat);
      if (!s.ok()) return s;
      if (st.load.tensor == tsid) return err(AMAP_EINVAL, "a statement reads the tensor it writes");
      lview = T[st.load.tensor];
      if (lflat) {
        lview.shape = {T[st.load.tensor].numel};
        lview.stride = {1};
      }
    }
    if (empty) continue;

    Piece R;
    R.ext.assign(st.bounds, st.bounds + n);
    R.fill = (es >= 8) ? st.fill_bits : (st.fill_bits & ((1ull << (8 * es)) - 1));
    RawStore rs;
    for (size_t d = 0; d < srow.row.size(); ++d) {
      int64_t lo, hi;
      aff_range(srow.row[d], R.ext, &lo, &hi);
      if (lo < 0 || hi >= sview.shape[d]) return err(AMAP_EOOB, "a store can leave its tensor");
      rs.lo.push_back(lo);
      rs.hi.push_back(hi);
      int64_t step = 0;
      for (int k = 0; k < n; ++k)
        if (R.ext[k] > 1) step = std::gcd(step, std::llabs(srow.row[d].c[k]));
      if (step <= 1) {
        rs.step.push_back(1);
        rs.rem.push_back(0);
      } else {
        rs.step.push_back(step);
        rs.rem.push_back(((srow.row[d].c0 % step) + step) % step);
      }
    }
    if (!linearise(srow, sview, n, &R.dst)) return err(AMAP_EOVERFLOW, "store offset overflows");
    s = check_injective(R);
    if (!s.ok()) return s;
    rs.piece = R;
    rs.piece.srcoff.c.assign(n, 0);
    s = check_overlap(S[tsid], T[tsid], rs);
    if (!s.ok()) return s;
    S[tsid].stores.push_back(rs);
    S[tsid].defined_points += box_points(R);

    if (is_const) {
      R.src = AMAP_CONST;
      R.srcoff.c.assign(n, 0);
      S[tsid].defs.push_back(R);
      continue;
    }
    const int tl = st.load.tensor;
    for (size_t d = 0; d < lrow.row.size(); ++d) {
      int64_t lo, hi;
      aff_range(lrow.row[d], R.ext, &lo, &hi);
      if (lo >= 0 && hi < lview.shape[d]) continue;
      if (!st.guarded) return err(AMAP_EOOB, "an unguarded load can leave its tensor");
      Con g;
      g.e = lrow.row[d];
      g.extent = lview.shape[d];
      R.guards.push_back(g);
    }
    R.src = tl;
    if (!linearise(lrow, lview, n, &R.srcoff)) return err(AMAP_EOVERFLOW, "load offset overflows");
    if (T[tl].input_slot < 0 && (flags & AMAP_COMPOSE_NO_FUSE)) {
      s = materialise(tl);
      if (!s.ok()) return s;
    }
    if (T[tl].input_slot >= 0) {
      if (tighten(R)) S[tsid].defs.push_back(R);
      continue;
    }
    if (S[tl].defs.empty() && T[tl].numel > 0)
      return err(AMAP_EUNDEFINED, "a statement reads a tensor that no earlier statement writes");
    s = compose_reader(R, S[tl], T[tl], es, (flags & AMAP_COMPOSE_QUASI_AFFINE) ? 1 : (flags & AMAP_COMPOSE_NO_QUASI_AFFINE) ? -1 : 0,
                       &S[tsid].defs);
    if (s.code == AMAP_EUNSUPPORTED) {
      // This pair cannot be eliminated (the paper's Section 3 also reports a pair that stays): keep t_l as a
      // temporary written by a stage of its own and read it like an input from here on.
      const Status m = materialise(tl);
      if (!m.ok()) return s;
      if (tighten(R)) S[tsid].defs.push_back(R);
      continue;
    }
    if (!s.ok()) return s;
  }

  // the outputs' definitions are the last stage: no output depends on another (a tensor that is an output and is
  // read again was composed through), so their pieces may run side by side
  std::vector<Piece> last;
  for (size_t k = 0; k < outputs.size(); ++k) {
    out->out_numels.push_back(T[outputs[k]].numel);
    Status s = close_tensor(outputs[k], -1, (int)k, &last);
    if (!s.ok()) return s;
  }
  out->out_numel = out->out_numels[0];
  StageInfo st;
  st.first_piece = (int)out->pieces.size();
  st.n_pieces = (int)last.size();
  st.dst_temp = -1;
  st.numel = out->out_numel;
  out->stages.push_back(st);
  out->pieces.insert(out->pieces.end(), last.begin(), last.end());
  return Status();
}

int64_t piece_unique_reads(const Piece &p, int64_t in_numel) { return unique_reads(p, in_numel); }

}  // namespace amap

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
using namespace amap;

static void log_map(const Map &m) {
  for (size_t q = 0; q < m.pieces.size(); ++q) {
    const Piece &p = m.pieces[q];
    fprintf(stderr, "[amap] piece %zu: input %d loops", q, p.src);
    for (int k = 0; k < p.n(); ++k)
      fprintf(stderr, " (%lld: src %lld dst %lld)", (long long)p.ext[k], (long long)(p.src == AMAP_CONST ? 0 : p.srcoff.c[k]),
              (long long)p.dst.c[k]);
    fprintf(stderr, " b_l %lld b_s %lld guards %zu domain %zu%s\n", (long long)p.srcoff.c0, (long long)p.dst.c0, p.guards.size(),
            p.domain.size(), p.qa.on ? " quasi-affine" : "");
  }
}

extern "C" int amap_compose(const amap_chain *chain, amap_map **out_map) { return amap_compose_ex(chain, 0, out_map); }

extern "C" int amap_compose_ex(const amap_chain *chain, uint32_t flags, amap_map **out_map) {
  if (!chain) return AMAP_EINVAL;
  return amap_compose_multi(chain, 1, &chain->output, flags, out_map);
}

extern "C" int amap_compose_multi(const amap_chain *chain, int32_t n_outputs, const int32_t *outputs, uint32_t flags,
                                  amap_map **out_map) {
  if (!out_map || !outputs || n_outputs < 1 ||
      (flags & ~(uint32_t)(AMAP_COMPOSE_NO_FUSE | AMAP_COMPOSE_QUASI_AFFINE | AMAP_COMPOSE_NO_QUASI_AFFINE)))
    return AMAP_EINVAL;
  amap_map *m = new (std::nothrow) amap_map();
  if (!m) return AMAP_ENOMEM;
  Status s;
  try {
    s = compose_chain(chain, std::vector<int>(outputs, outputs + n_outputs), flags, &m->m);
  } catch (const std::bad_alloc &) {
    s.code = AMAP_ENOMEM;
  }
  if (!s.ok()) {
    if (log_enabled()) fprintf(stderr, "[amap] compose failed: %s\n", s.msg.c_str());
    delete m;
    return s.code;
  }
  Map &mm = m->m;
  mm.guard_views.resize(mm.pieces.size());
  mm.domain_views.resize(mm.pieces.size());
  for (size_t q = 0; q < mm.pieces.size(); ++q) {
    for (auto &g : mm.pieces[q].guards) mm.guard_views[q].push_back({g.e.c.data(), g.e.c0, g.extent});
    for (auto &g : mm.pieces[q].domain) mm.domain_views[q].push_back({g.e.c.data(), g.e.c0, g.extent});
  }
  if (log_enabled()) log_map(mm);
  *out_map = m;
  return AMAP_OK;
}

extern "C" void amap_map_destroy(amap_map *map) { delete map; }

extern "C" int amap_map_num_pieces(const amap_map *map, int32_t *n) {
  if (!map || !n) return AMAP_EINVAL;
  *n = (int32_t)map->m.pieces.size();
  return AMAP_OK;
}

extern "C" int amap_map_get_piece(const amap_map *map, int32_t k, amap_piece *out) {
  if (!map || !out || k < 0 || k >= (int32_t)map->m.pieces.size()) return AMAP_EINVAL;
  const Piece &p = map->m.pieces[k];
  out->n_loops = p.n();
  out->bounds = p.ext.data();
  out->input = p.src;
  out->C_l = (p.src == AMAP_CONST) ? nullptr : p.srcoff.c.data();
  out->b_l = (p.src == AMAP_CONST) ? 0 : p.srcoff.c0;
  out->C_s = p.dst.c.data();
  out->b_s = p.dst.c0;
  out->n_guards = (int32_t)p.guards.size();
  out->guards = map->m.guard_views[k].data();
  out->n_domain = (int32_t)p.domain.size();
  out->domain = map->m.domain_views[k].data();
  out->fill_bits = p.fill;
  out->output = p.out;
  const bool qa = p.src != AMAP_CONST && p.qa.on;
  out->n_digits = qa ? (int32_t)p.qa.radix.size() : 0;
  out->digit_radix = qa ? p.qa.radix.data() : nullptr;
  out->digit_stride = qa ? p.qa.stride.data() : nullptr;
  out->F = qa ? p.qa.f.c.data() : nullptr;
  out->f0 = qa ? p.qa.f.c0 : 0;
  return AMAP_OK;
}

extern "C" int amap_map_num_outputs(const amap_map *map, int32_t *n) {
  if (!map || !n) return AMAP_EINVAL;
  *n = (int32_t)map->m.out_numels.size();
  return AMAP_OK;
}

extern "C" int amap_map_output_numel(const amap_map *map, int32_t k, int64_t *numel) {
  if (!map || !numel || k < 0 || k >= (int32_t)map->m.out_numels.size()) return AMAP_EINVAL;
  *numel = map->m.out_numels[k];
  return AMAP_OK;
}

extern "C" int amap_map_num_stages(const amap_map *map, int32_t *n) {
  if (!map || !n) return AMAP_EINVAL;
  *n = (int32_t)map->m.stages.size();
  return AMAP_OK;
}

extern "C" int amap_map_get_stage(const amap_map *map, int32_t s, int32_t *first_piece, int32_t *n_pieces, int32_t *dst_temp,
                                  int64_t *dst_numel) {
  if (!map || s < 0 || s >= (int32_t)map->m.stages.size()) return AMAP_EINVAL;
  const StageInfo &st = map->m.stages[s];
  if (first_piece) *first_piece = st.first_piece;
  if (n_pieces) *n_pieces = st.n_pieces;
  if (dst_temp) *dst_temp = st.dst_temp;
  if (dst_numel) *dst_numel = st.numel;
  return AMAP_OK;
}

extern "C" int amap_map_sizes(const amap_map *map, int32_t *n_inputs, int64_t *in_numel, int64_t *out_numel,
                              int32_t *elem_size) {
  if (!map) return AMAP_EINVAL;
  if (n_inputs) *n_inputs = (int32_t)map->m.in_numel.size();
  if (in_numel)
    for (size_t q = 0; q < map->m.in_numel.size(); ++q) in_numel[q] = map->m.in_numel[q];
  if (out_numel) *out_numel = map->m.out_numel;
  if (elem_size) *elem_size = map->m.elem_size;
  return AMAP_OK;
}

extern "C" int amap_map_device_view(const amap_map *map, amap_device_view *out) {
  if (!map || !out) return AMAP_EINVAL;
  const Map &m = map->m;
  if (m.stages.size() != 1 || m.out_numels.size() > 1) return AMAP_EUNSUPPORTED;
  if (m.pieces.size() > (size_t)AMAP_VIEW_MAX_PIECES) return AMAP_ETOOLARGE;
  memset(out, 0, sizeof *out);
  out->n_pieces = (int32_t)m.pieces.size();
  out->elem_size = m.elem_size;
  out->n_inputs = (int32_t)m.in_numel.size();
  out->out_numel = m.out_numel;
  for (size_t q = 0; q < m.pieces.size(); ++q) {
    const Piece &p = m.pieces[q];
    amap_view_piece &v = out->piece[q];
    if (p.n() > AMAP_VIEW_MAX_LOOPS || p.guards.size() + p.domain.size() > (size_t)AMAP_VIEW_MAX_CONS) return AMAP_ETOOLARGE;
    if (p.src != AMAP_CONST && p.qa.on) return AMAP_EUNSUPPORTED;  // the view holds affine pieces only
    // canonical pieces have positive destination strides in descending order; decoding an output index digit by
    // digit also needs them nested
    for (int k = 0; k < p.n(); ++k)
      if (p.dst.c[k] <= 0 || (k > 0 && p.dst.c[k] > p.dst.c[k - 1])) return AMAP_EUNSUPPORTED;
    if (!nested_strides(p.dst.c, p.ext)) return AMAP_EUNSUPPORTED;
    v.n_loops = p.n();
    v.input = p.src;
    v.n_guards = (int32_t)p.guards.size();
    v.n_domain = (int32_t)p.domain.size();
    v.b_s = p.dst.c0;
    v.b_l = p.src == AMAP_CONST ? 0 : p.srcoff.c0;
    v.fill_bits = p.fill;
    for (int k = 0; k < p.n(); ++k) {
      v.ext[k] = p.ext[k];
      v.dst_stride[k] = p.dst.c[k];
      v.src_stride[k] = p.src == AMAP_CONST ? 0 : p.srcoff.c[k];
    }
    int c = 0;
    auto put = [&](const Con &g) {
      for (int k = 0; k < p.n(); ++k) v.cons[c].coef[k] = g.e.c[k];
      v.cons[c].offset = g.e.c0;
      v.cons[c].extent = g.extent;
      ++c;
    };
    for (auto &g : p.guards) put(g);
    for (auto &g : p.domain) put(g);
    for (int k = 0; k < p.n(); ++k) {  // division by the destination strides as multiply-and-shift (32-bit path)
      const uint64_t d = (uint64_t)std::min<int64_t>(p.dst.c[k], 0xFFFFFFFFll);
      uint32_t l = 0;
      while (l < 32 && (1ull << l) < d) ++l;
      v.fd_mul[k] = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
      v.fd_sh1[k] = (uint8_t)(l < 1 ? l : 1);
      v.fd_sh2[k] = (uint8_t)(l < 1 ? 0 : l - 1);
    }
  }
  // The 32-bit path is valid when nothing the functor computes can leave 31 bits: output and input sizes, and the
  // range of every constraint expression over its piece's box.
  bool small = m.out_numel < (1ll << 31);
  for (int64_t n : m.in_numel) small = small && n < (1ll << 31);
  for (const Piece &p : m.pieces) {
    auto fits = [&](const Aff &a) {
      int64_t lo, hi;
      aff_range(a, p.ext, &lo, &hi);
      __int128 span = std::llabs(a.c0);
      for (int k = 0; k < p.n(); ++k) span += (__int128)std::llabs(a.c[k]) * (p.ext[k] - 1);
      return span < (1ll << 31) && lo > -(1ll << 31) && hi < (1ll << 31);
    };
    for (auto &g : p.guards) small = small && fits(g.e) && g.extent < (1ll << 31);
    for (auto &g : p.domain) small = small && fits(g.e);
    for (int k = 0; k < p.n(); ++k) small = small && p.ext[k] < (1ll << 31) && p.dst.c[k] < (1ll << 31);
  }
  out->small = small ? 1 : 0;
  return AMAP_OK;
}

extern "C" const char *amap_strerror(int code) {
  switch (code) {
    case AMAP_OK: return "ok";
    case AMAP_EINVAL: return "invalid argument";
    case AMAP_ESTORE_NOT_INJECTIVE: return "a store map is not injective and has no reverse";
    case AMAP_EOOB: return "an unguarded access can leave its tensor";
    case AMAP_EUNDEFINED: return "an element that is read or returned is never written";
    case AMAP_EOVERLAP: return "two statements write the same element";
    case AMAP_EOVERFLOW: return "an offset or size overflows";
    case AMAP_EALIGN: return "a device pointer is not aligned as the plan requires";
    case AMAP_ECUDA: return "a CUDA call failed";
    case AMAP_EUNSUPPORTED: return "the maps cannot be composed affinely by this library";
    case AMAP_ENOMEM: return "out of memory";
    case AMAP_ETOOLARGE: return "the plan has more descriptors than the fixed table of amap_execute_static holds";
  }
  return "unknown amap status";
}
