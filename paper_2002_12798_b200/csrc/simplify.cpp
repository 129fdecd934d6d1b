// Loop-nest housekeeping for composed pieces: interval analysis, clipping of
// constraints into the loop box, point counting, and the canonical form the
// planner consumes (unit loops dropped, loops ordered by destination stride,
// adjacent loops merged when both sides and every constraint allow it).
// The access maps stay in the paper's form f(i) = C i + b with constant C, b
// (Section 2); only the loop nest that parameterises them is rewritten.
#include <algorithm>
#include <cstdlib>
#include <numeric>

#include "amap_internal.hpp"

namespace amap {

static inline int64_t floordiv(int64_t a, int64_t b) {
  int64_t q = a / b, r = a % b;
  return (r != 0 && ((r < 0) != (b < 0))) ? q - 1 : q;
}
static inline int64_t ceildiv(int64_t a, int64_t b) { return -floordiv(-a, b); }

void aff_range(const Aff &a, const std::vector<int64_t> &ext, int64_t *lo, int64_t *hi) {
  __int128 l = a.c0, h = a.c0;
  for (size_t k = 0; k < ext.size(); ++k) {
    __int128 v = (__int128)a.c[k] * (ext[k] - 1);
    if (v > 0) h += v; else l += v;
  }
  const __int128 big = (__int128)INT64_MAX / 2;
  *lo = (int64_t)std::max<__int128>(l, -big);
  *hi = (int64_t)std::min<__int128>(h, big);
}

template <class F>
static void for_each_aff(Piece &p, F f) {
  f(p.dst);
  if (p.src != AMAP_CONST) f(p.srcoff);
  if (p.src != AMAP_CONST && p.qa.on) f(p.qa.f);
  for (auto &g : p.guards) f(g.e);
  for (auto &g : p.domain) f(g.e);
}

void reverse_loop(Piece &p, int k) {
  const int64_t last = p.ext[k] - 1;
  for_each_aff(p, [&](Aff &a) {
    a.c0 += a.c[k] * last;
    a.c[k] = -a.c[k];
  });
}

void permute_loops(Piece &p, const std::vector<int> &order) {
  auto perm = [&](std::vector<int64_t> &v) {
    std::vector<int64_t> w(order.size());
    for (size_t k = 0; k < order.size(); ++k) w[k] = v[order[k]];
    v.swap(w);
  };
  perm(p.ext);
  if (p.src == AMAP_CONST) p.srcoff.c.assign(order.size(), 0);
  for_each_aff(p, [&](Aff &a) { perm(a.c); });
}

static void erase_loop(Piece &p, int k) {
  p.ext.erase(p.ext.begin() + k);
  if (p.src == AMAP_CONST && (int)p.srcoff.c.size() > k) p.srcoff.c.erase(p.srcoff.c.begin() + k);
  for_each_aff(p, [&](Aff &a) { a.c.erase(a.c.begin() + k); });
}

void drop_unit_loops(Piece &p) {
  for (int k = p.n() - 1; k >= 0; --k)
    if (p.ext[k] == 1) erase_loop(p, k);
}

// restrict loop k to [lo, lo+len)
static void clip_loop(Piece &p, int k, int64_t lo, int64_t len) {
  for_each_aff(p, [&](Aff &a) { a.c0 += a.c[k] * lo; });
  p.ext[k] = len;
}

// loops with more than one iteration that the expression depends on
static int involved(const Aff &a, const std::vector<int64_t> &ext, int *which) {
  int cnt = 0;
  for (size_t k = 0; k < ext.size(); ++k)
    if (a.c[k] != 0 && ext[k] > 1) {
      ++cnt;
      *which = (int)k;
    }
  return cnt;
}

// range of i_k for which 0 <= c0 + a*i_k < extent, intersected with the box
static void valid_range(const Con &g, int k, int64_t ek, int64_t *lo, int64_t *hi) {
  const int64_t a = g.e.c[k];
  int64_t c0 = g.e.c0;  // other involved loops have extent 1 -> contribute 0
  int64_t l, h;
  if (a > 0) {
    l = ceildiv(-c0, a);
    h = floordiv(g.extent - 1 - c0, a);
  } else {
    l = ceildiv(g.extent - 1 - c0, a);
    h = floordiv(-c0, a);
  }
  *lo = std::max<int64_t>(l, 0);
  *hi = std::min<int64_t>(h, ek - 1);
}

bool tighten(Piece &p) {
  for (int64_t e : p.ext)
    if (e <= 0) return false;
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t q = 0; q < p.domain.size();) {
      Con &g = p.domain[q];
      int64_t lo, hi;
      aff_range(g.e, p.ext, &lo, &hi);
      if (hi < 0 || lo >= g.extent) return false;
      if (lo >= 0 && hi < g.extent) {
        p.domain.erase(p.domain.begin() + q);
        continue;
      }
      int k = -1;
      if (involved(g.e, p.ext, &k) == 1) {
        int64_t l, h;
        valid_range(g, k, p.ext[k], &l, &h);
        if (l > h) return false;
        clip_loop(p, k, l, h - l + 1);
        p.domain.erase(p.domain.begin() + q);
        changed = true;
        continue;
      }
      ++q;
    }
    for (size_t q = 0; q < p.guards.size();) {
      Con &g = p.guards[q];
      int64_t lo, hi;
      aff_range(g.e, p.ext, &lo, &hi);
      if (hi < 0 || lo >= g.extent) {  // never loads: a pure fill piece
        p.src = AMAP_CONST;
        p.srcoff = Aff();
        p.srcoff.c.assign(p.ext.size(), 0);
        p.qa = QuasiSrc();
        p.guards.clear();
        break;
      }
      if (lo >= 0 && hi < g.extent) {
        p.guards.erase(p.guards.begin() + q);
        continue;
      }
      ++q;
    }
  }
  return true;
}

int64_t count_points(const Piece &p0) {
  Piece p = p0;
  if (!tighten(p)) return 0;
  std::vector<int> loops;  // loops some remaining domain constraint depends on
  std::vector<char> in(p.ext.size(), 0);
  for (auto &g : p.domain)
    for (size_t k = 0; k < p.ext.size(); ++k)
      if (g.e.c[k] != 0 && p.ext[k] > 1 && !in[k]) {
        in[k] = 1;
        loops.push_back((int)k);
      }
  __int128 free_pts = 1;
  for (size_t k = 0; k < p.ext.size(); ++k)
    if (!in[k]) free_pts *= p.ext[k];
  __int128 combos = 1;
  for (int k : loops) {
    combos *= p.ext[k];
    if (combos > 50000000) return -1;
  }
  int64_t good = 0;
  std::vector<int64_t> idx(loops.size(), 0);
  for (int64_t t = 0; t < (int64_t)combos; ++t) {
    bool ok = true;
    for (auto &g : p.domain) {
      int64_t v = g.e.c0;
      for (size_t q = 0; q < loops.size(); ++q) v += g.e.c[loops[q]] * idx[q];
      if (v < 0 || v >= g.extent) {
        ok = false;
        break;
      }
    }
    good += ok;
    for (int q = (int)loops.size() - 1; q >= 0; --q) {
      if (++idx[q] < p.ext[loops[q]]) break;
      idx[q] = 0;
    }
  }
  __int128 total = free_pts * good;
  if (total > INT64_MAX / 2) return -1;
  return (int64_t)total;
}

// ---------------------------------------------------------------------------
static bool mergeable(const Piece &p, int k) {  // loops k and k+1
  const int64_t e = p.ext[k + 1];
  auto fits = [&](const Aff &a) { return a.c[k] == e * a.c[k + 1]; };
  if (!fits(p.dst)) return false;
  if (p.src != AMAP_CONST && !fits(p.srcoff)) return false;
  if (p.src != AMAP_CONST && p.qa.on && !fits(p.qa.f)) return false;
  for (auto &g : p.guards)
    if (!fits(g.e)) return false;
  for (auto &g : p.domain)
    if (!fits(g.e)) return false;
  return true;
}

static void canonical_loops(Piece &p) {
  drop_unit_loops(p);
  for (int k = 0; k < p.n(); ++k)
    if (p.dst.c[k] < 0) reverse_loop(p, k);
  std::vector<int> order(p.n());
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return p.dst.c[a] > p.dst.c[b]; });
  permute_loops(p, order);
  for (int k = 0; k + 1 < p.n();) {
    if (mergeable(p, k)) {
      p.ext[k + 1] *= p.ext[k];
      erase_loop(p, k);
      if (k > 0) --k;
    } else {
      ++k;
    }
  }
}

// Two unconstrained fill pieces of the same value whose boxes touch along one loop (same strides, same other
// extents, the second starting where the first ends) are one box; repeated to the fixpoint, this turns the
// per-operand border slabs of a padded concat into a few long runs.
static bool try_merge_fill(Piece &a, const Piece &b) {
  if (a.src != AMAP_CONST || b.src != AMAP_CONST || a.fill != b.fill) return false;
  if (!a.guards.empty() || !a.domain.empty() || !b.guards.empty() || !b.domain.empty()) return false;
  if (a.n() != b.n() || a.dst.c != b.dst.c) return false;
  int diff = -1;
  for (int k = 0; k < a.n(); ++k)
    if (a.ext[k] != b.ext[k]) {
      if (diff >= 0) return false;
      diff = k;
    }
  const int64_t delta = b.dst.c0 - a.dst.c0;
  for (int k = 0; k < a.n(); ++k) {
    if (diff >= 0 && k != diff) continue;
    if (delta == a.ext[k] * a.dst.c[k]) {
      a.ext[k] += b.ext[k];
      return true;
    }
  }
  return false;
}

static void merge_fill_pieces(std::vector<Piece> &pieces) {
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t i = 0; i < pieces.size() && !changed; ++i)
      for (size_t j = 0; j < pieces.size() && !changed; ++j) {
        if (i == j || !try_merge_fill(pieces[i], pieces[j])) continue;
        pieces.erase(pieces.begin() + j);
        Piece &p = pieces[j < i ? i - 1 : i];
        canonical_loops(p);  // the longer loop may now merge with its neighbour
        changed = true;
      }
  }
}

int64_t piece_run_elems(const Piece &p, int in, int64_t cap) {
  if (in < 0 || in >= p.n() || p.dst.c[in] != 1) return 1;
  for (auto &g : p.guards)
    if (g.e.c[in] != 0) return 1;
  for (auto &g : p.domain)
    if (g.e.c[in] != 0) return 1;
  if (p.src == AMAP_CONST) return 1;
  auto divides = [](int64_t q, int64_t v) { return v % q == 0; };
  int64_t q = 1;
  while (q * 2 <= cap) q *= 2;
  for (; q > 1; q /= 2) {
    bool ok = divides(q, p.ext[in]) && divides(q, p.dst.c0);
    for (int k = 0; k < p.n() && ok; ++k)
      if (k != in) ok = divides(q, p.dst.c[k]);
    if (!p.qa.on) {
      ok = ok && p.srcoff.c[in] == 1 && divides(q, p.srcoff.c0);
      for (int k = 0; k < p.n() && ok; ++k)
        if (k != in) ok = divides(q, p.srcoff.c[k]);
    } else {
      // the run walks f by one; it stays inside one innermost digit and that digit is contiguous in the source
      const size_t K = p.qa.radix.size();
      ok = ok && K > 0 && p.qa.f.c[in] == 1 && divides(q, p.qa.f.c0) && p.qa.stride[K - 1] == 1 &&
           divides(q, p.qa.radix[K - 1]) && divides(q, p.srcoff.c0);
      for (int k = 0; k < p.n() && ok; ++k)
        if (k != in) ok = divides(q, p.qa.f.c[k]);
      for (size_t d = 0; d + 1 < K && ok; ++d) ok = divides(q, p.qa.stride[d]);
    }
    if (ok) return q;
  }
  return 1;
}

Status canonicalise(std::vector<Piece> &pieces) {
  std::vector<Piece> work;
  work.swap(pieces);
  while (!work.empty()) {
    Piece p = std::move(work.back());
    work.pop_back();
    if (!tighten(p)) continue;
    // a guard that depends on one loop only splits the box into a copy part and fill slabs
    int gi = -1, gk = -1;
    for (size_t q = 0; q < p.guards.size() && gi < 0; ++q) {
      int k = -1;
      if (involved(p.guards[q].e, p.ext, &k) == 1) {
        gi = (int)q;
        gk = k;
      }
    }
    if (gi < 0) {
      canonical_loops(p);
      pieces.push_back(std::move(p));
      continue;
    }
    int64_t lo, hi;
    valid_range(p.guards[gi], gk, p.ext[gk], &lo, &hi);
    const int64_t ek = p.ext[gk];
    auto fill_part = [&](int64_t from, int64_t len) {
      if (len <= 0) return;
      Piece f = p;
      f.src = AMAP_CONST;
      f.srcoff = Aff();
      f.srcoff.c.assign(f.ext.size(), 0);
      f.qa = QuasiSrc();
      f.guards.clear();
      clip_loop(f, gk, from, len);
      work.push_back(std::move(f));
    };
    if (lo > hi) {  // the guard never holds
      fill_part(0, ek);
      continue;
    }
    fill_part(0, lo);
    fill_part(hi + 1, ek - 1 - hi);
    Piece mid = p;
    mid.guards.erase(mid.guards.begin() + gi);
    clip_loop(mid, gk, lo, hi - lo + 1);
    work.push_back(std::move(mid));
  }
  merge_fill_pieces(pieces);
  // The kernels index a piece's items with 32 bits: cut pieces of 2^31 points or more in two along their
  // outermost loop until every piece is smaller.
  for (size_t q = 0; q < pieces.size();) {
    __int128 pts = 1;
    for (int64_t e : pieces[q].ext) pts *= e;
    if (pts < ((__int128)1 << 31) || pieces[q].n() == 0) {
      ++q;
      continue;
    }
    Piece lo = pieces[q], hi = pieces[q];
    const int64_t half = lo.ext[0] / 2;
    clip_loop(lo, 0, 0, half);
    clip_loop(hi, 0, half, hi.ext[0] - half);
    canonical_loops(lo);
    canonical_loops(hi);
    pieces[q] = lo;
    pieces.insert(pieces.begin() + q + 1, hi);
  }
  // deterministic order: by destination offset
  std::stable_sort(pieces.begin(), pieces.end(), [](const Piece &a, const Piece &b) { return a.dst.c0 < b.dst.c0; });
  return Status();
}

}  // namespace amap
