// amap_plan / amap_execute: classify the pieces of a composed map, build the
// device descriptor table and enqueue the copy kernel(s).
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "amap_internal.hpp"
#include "kernels.cuh"

namespace amap {
int64_t piece_unique_reads(const Piece &p, int64_t in_numel);
}
using namespace amap;

static thread_local std::string g_cuda_error;

static int cuda_fail(cudaError_t e, const char *what) {
  g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
  return AMAP_ECUDA;
}
#define CUDA_TRY(expr)                                  \
  do {                                                  \
    cudaError_t e_ = (expr);                            \
    if (e_ != cudaSuccess) return cuda_fail(e_, #expr); \
  } while (0)

extern "C" const char *amap_last_cuda_error(void) { return g_cuda_error.c_str(); }

struct Launch {
  int kind;  // DevKind
  int unit;  // bytes per item (affine kernel) / element size (transpose kernel)
  int cons;  // affine / strip kernel: constraint slots evaluated per unit (0, 2 or kDevMaxCons)
             // transpose kernel: bytes per global access (16, 8, 4, 2), 0 for the shifted-row kernel, -1 for the
             // realigning kernel, -2 for the flat-destination kernel, -3 for the flat-source kernel
  int wide;  // affine kernel: 1 when a byte offset can reach 4 GiB (64-bit offsets)
  int first_piece;
  int n_pieces;
  uint32_t n_blocks;
  int stage;  // which stage of the map this launch belongs to
  int threads = 0;  // flat transposes only: block size and dynamic shared memory of the launch
  int smem = 0;
  int paired = 0;   // flat-destination transpose of 2-byte elements: every piece's rows are an even number of elements long
};

struct amap_plan_t {
  int device = 0;
  int elem_size = 0;
  int pointer_align = 0;
  bool pdl = true;  // launch with programmatic stream serialisation
  std::vector<int64_t> in_numel;
  std::vector<char> in_used;        // per input: some piece reads it (the pointer of an unused input may be null)
  int64_t out_numel = 0;            // output 0
  std::vector<int64_t> out_numels;  // every output
  std::vector<int64_t> temp_numel;  // temporaries between stages
  std::vector<int> stage_dst;       // per stage: temporary written, -1 = the output
  std::vector<void *> temps;        // device memory of the temporaries (owned)
  std::vector<DevPiece> table;
  std::vector<int> piece_kernel;  // amap_kernel_kind per map piece
  std::vector<Launch> launches;
  std::vector<LaunchDesc> launch_desc;  // per launch; n_pieces == 0 when it has too many pieces for the parameters
  DevPiece *dev_table = nullptr;
  amap_stats stats;
  // staging for amap_execute_host (allocated on first use)
  std::vector<void *> stage_in;
  void *stage_out = nullptr;
  // amap_execute_host pipelines batch slabs when every piece's outermost loop is one batch loop that cuts the
  // inputs and the output into independent slabs: a second plan for one slab, run once per slab
  amap_plan_t *slab_plan = nullptr;
  int n_slabs = 0;
  std::vector<int64_t> slab_in_bytes;
  int64_t slab_out_bytes = 0;
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  std::vector<cudaEvent_t> events;  // [0] start, then per slab: input ready, kernel done; last: output done
};

static FastDiv make_fastdiv(uint32_t d) {
  FastDiv f;
  f.d = d;
  uint32_t l = 0;
  while (l < 32 && (1ull << l) < d) ++l;  // ceil(log2 d)
  f.mul = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
  f.sh1 = l < 1 ? l : 1;
  f.sh2 = l < 1 ? 0 : l - 1;
  return f;
}

static const int kDefaultSms = 148;  // B200; only dry plans rely on it
static const int kUnroll = kStrip;  // units per thread in the affine kernel

// largest power-of-two unit (<= 16 bytes) in which the piece is still an affine loop nest
static int pick_unit(const Piece &p, int es, int ptr_align, int force_kind) {
  if (force_kind == AMAP_KERNEL_GATHER) return es;
  const int n = p.n();
  if (n == 0) return es;
  const int in = n - 1;  // canonical order: innermost destination loop last
  if (p.src != AMAP_CONST && p.qa.on) {  // quasi-affine: as wide as the run that shares one digit decomposition
    const int64_t q = piece_run_elems(p, in, 16 / es);
    int V = (int)(q * es);
    while (V > es && V > ptr_align) V >>= 1;
    return V;
  }
  if (p.dst.c[in] != 1) return es;
  if (p.src != AMAP_CONST && p.srcoff.c[in] != 1) return es;
  for (auto &g : p.guards)
    if (g.e.c[in] != 0) return es;
  for (auto &g : p.domain)
    if (g.e.c[in] != 0) return es;
  for (int V = 16; V > es; V >>= 1) {
    if (V > ptr_align) continue;
    const int64_t q = V / es;  // elements per unit
    bool ok = (p.ext[in] % q == 0) && (p.dst.c0 % q == 0) && (p.src == AMAP_CONST || p.srcoff.c0 % q == 0);
    for (int k = 0; k < in && ok; ++k) {
      if (p.dst.c[k] % q) ok = false;
      if (p.src != AMAP_CONST && p.srcoff.c[k] % q) ok = false;
    }
    if (ok) return V;
  }
  return es;
}

static uint64_t replicate_fill(uint64_t fill, int es) {
  if (es >= 8) return fill;
  uint64_t v = 0;
  for (int b = 0; b < 8; b += es) v |= (fill & ((1ull << (8 * es)) - 1)) << (8 * b);
  return v;
}

static int build_affine_piece(const Piece &p, int es, int V, DevPiece *d) {
  memset(d, 0, sizeof *d);
  d->kind = kDevAffine;
  d->input = p.src;
  d->out = p.out;
  d->unit_bytes = V;
  d->fill[0] = replicate_fill(p.fill, es);
  d->fill[1] = (es == 16) ? 0 : d->fill[0];
  d->soff = (p.src == AMAP_CONST) ? 0 : p.srcoff.c0 * es;
  d->doff = p.dst.c0 * es;
  const int q = V / es;
  std::vector<int> loops;
  for (int k = 0; k < p.n(); ++k) {
    int64_t e = p.ext[k];
    if (k == p.n() - 1) e /= q;  // the innermost loop counts units
    if (e == 1) continue;
    loops.push_back(k);
  }
  if ((int)loops.size() > kDevMaxLoops) return AMAP_EUNSUPPORTED;
  if ((int)(p.guards.size() + p.domain.size()) > kDevMaxCons) return AMAP_EUNSUPPORTED;
  d->n_loops = (int)loops.size();
  unsigned __int128 items = 1;
  for (size_t j = 0; j < loops.size(); ++j) {
    const int k = loops[j];
    int64_t e = p.ext[k];
    if (k == p.n() - 1) e /= q;
    d->ext[j] = (uint32_t)e;
    d->fd[j] = make_fastdiv((uint32_t)e);
    const int64_t unit = (k == p.n() - 1) ? V : es;  // the innermost loop steps by whole units
    d->sstride[j] = (p.src == AMAP_CONST) ? 0 : p.srcoff.c[k] * unit;
    d->dstride[j] = p.dst.c[k] * unit;
    items *= (uint64_t)e;
  }
  if (items >= (1ull << 32) - (uint64_t)kAffineThreads * kUnroll) return AMAP_EUNSUPPORTED;
  d->n_items = (uint64_t)items;
  if (p.src != AMAP_CONST && p.qa.on) {
    const int K = (int)p.qa.radix.size();
    if (K < 1 || K > kQuasiMaxDigits || p.qa.radix[K - 1] % q) return AMAP_EUNSUPPORTED;
    int64_t lo, hi;
    aff_range(p.qa.f, p.ext, &lo, &hi);
    if (hi >= (1ll << 32) || lo <= -(1ll << 31)) return AMAP_EUNSUPPORTED;  // 32-bit arithmetic in the kernel
    d->qa_n = K;
    d->qa_f0 = (uint32_t)(p.qa.f.c0 / q);
    for (size_t j = 0; j < loops.size(); ++j) {
      const int k = loops[j];
      d->qa_fstride[j] = (k == p.n() - 1 && q > 1) ? 1u : (uint32_t)(p.qa.f.c[k] / q);
    }
    for (int t = 0; t < K; ++t) {
      const int64_t radix = (t == K - 1) ? p.qa.radix[t] / q : p.qa.radix[t];
      if (radix < 1 || radix >= (1ll << 32)) return AMAP_EUNSUPPORTED;
      d->qa_radix[t] = (uint32_t)radix;
      d->qa_fd[t] = make_fastdiv((uint32_t)radix);
      d->qa_stride[t] = p.qa.stride[t] * ((t == K - 1) ? (int64_t)V : (int64_t)es);
    }
  }
  d->n_guards = (int)p.guards.size();
  d->n_domain = (int)p.domain.size();
  int c = 0;
  // the kernel evaluates constraints in 32-bit arithmetic: every partial sum must fit
  auto put = [&](const Con &g) -> bool {
    int64_t span = std::llabs(g.e.c0);
    for (size_t j = 0; j < loops.size(); ++j) {
      const int64_t v = g.e.c[loops[j]];
      if (std::llabs(v) > INT32_MAX) return false;
      span += std::llabs(v) * (int64_t)(d->ext[j] - 1);
      d->cons[c].coef[j] = (int32_t)v;
    }
    if (span >= INT32_MAX) return false;
    d->cons[c].off = (int32_t)g.e.c0;
    d->cons[c].extent = (int32_t)std::min<int64_t>(g.extent, INT32_MAX);
    ++c;
    return true;
  };
  for (auto &g : p.guards)
    if (!put(g)) return AMAP_EOVERFLOW;
  for (auto &g : p.domain)
    if (!put(g)) return AMAP_EOVERFLOW;
  const uint64_t per_block = (uint64_t)kAffineThreads * kUnroll;
  d->n_blocks = (uint32_t)((d->n_items + per_block - 1) / per_block);
  return AMAP_OK;
}

// Turns an affine descriptor with two or more loops into a strip descriptor:
// picks the loop to walk (not the innermost; one whose extent is a multiple of
// kStrip if there is one, else the longest; the innermost such candidate) and
// rescales it to count strips.
static bool make_strip(DevPiece *d) {
  const int n = d->n_loops;
  if (n < 2) return false;
  int ku = -1;
  // a loop along which the source advances by less than a 32-byte sector: walking it makes a thread's loads
  // share sectors (element-wise gathers such as transposes with odd extents)
  if (d->input >= 0)
    for (int k = n - 2; k >= 0; --k)
      if (d->sstride[k] != 0 && std::llabs(d->sstride[k]) < 32 && d->ext[k] >= kStrip &&
          (ku < 0 || std::llabs(d->sstride[k]) < std::llabs(d->sstride[ku])))
        ku = k;
  if (ku < 0)
    for (int k = n - 2; k >= 0; --k)
      if (d->ext[k] % kStrip == 0) {
        ku = k;
        break;
      }
  if (ku < 0) {
    ku = n - 2;
    for (int k = n - 3; k >= 0; --k)
      if (d->ext[k] > d->ext[ku]) ku = k;
  }
  const int nc = d->n_guards + d->n_domain;
  for (int c = 0; c < nc; ++c)
    if (std::llabs((int64_t)d->cons[c].coef[ku]) * kStrip > INT32_MAX / 4) return false;
  d->kind = kDevStrip;
  d->ku = ku;
  d->ku_ext = d->ext[ku];
  d->ku_ss = d->sstride[ku];
  d->ku_ds = d->dstride[ku];
  for (int c = 0; c < nc; ++c) {
    d->ku_coef[c] = d->cons[c].coef[ku];
    d->cons[c].coef[ku] *= kStrip;
  }
  const uint32_t strips = (d->ext[ku] + kStrip - 1) / kStrip;
  d->ext[ku] = strips;
  d->fd[ku] = make_fastdiv(strips);
  d->sstride[ku] *= kStrip;
  d->dstride[ku] *= kStrip;
  uint64_t items = 1;
  for (int k = 0; k < n; ++k) items *= d->ext[k];
  d->n_items = items;
  d->n_blocks = (uint32_t)((items + kAffineThreads - 1) / kAffineThreads);
  return true;
}

// Walks a device descriptor on the HOST with the kernel's own arithmetic and
// checks every address it would form: inside its buffer and aligned to the
// unit.  Small pieces are walked completely, large ones at their first and
// last items and a pseudo-random sample.  A failure here is a planner bug and
// is reported instead of being launched.
static uint32_t host_fast_div(uint32_t n, const FastDiv &f) {
  const uint32_t t = (uint32_t)(((uint64_t)f.mul * n) >> 32);
  return (t + ((n - t) >> f.sh1)) >> f.sh2;
}

static bool check_affine_item(const DevPiece &d, uint64_t L, int64_t in_bytes, int64_t out_bytes) {
  uint32_t rem = (uint32_t)L;
  int64_t s = d.soff, o = d.doff;
  int64_t acc[kDevMaxCons] = {0};
  const int nc = d.n_guards + d.n_domain;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    const uint32_t q = host_fast_div(rem, d.fd[k]);
    if (q != rem / d.ext[k]) return false;
    const uint32_t i = rem - q * d.ext[k];
    rem = q;
    s += (int64_t)i * d.sstride[k];
    o += (int64_t)i * d.dstride[k];
    for (int c = 0; c < nc; ++c) acc[c] += (int64_t)d.cons[c].coef[k] * i;
  }
  if (rem != 0) return false;
  if (d.qa_n > 0) {  // the quasi-affine source offset, with the kernel's 32-bit arithmetic
    uint32_t r2 = (uint32_t)L, f = d.qa_f0;
    for (int k = d.n_loops - 1; k >= 0; --k) {
      const uint32_t q = r2 / d.ext[k];
      f += (r2 - q * d.ext[k]) * d.qa_fstride[k];
      r2 = q;
    }
    for (int t = d.qa_n - 1; t >= 0; --t) {
      const uint32_t q = host_fast_div(f, d.qa_fd[t]);
      if (q != f / d.qa_radix[t]) return false;
      s += (int64_t)(f - q * d.qa_radix[t]) * d.qa_stride[t];
      f = q;
    }
  }
  if (d.kind == kDevStrip) {  // walk the strip as the kernel does
    uint32_t r2 = (uint32_t)L, strip = 0;
    for (int k = d.n_loops - 1; k >= 0; --k) {
      const uint32_t q = r2 / d.ext[k];
      if (k == d.ku) strip = r2 - q * d.ext[k];
      r2 = q;
    }
    if ((uint64_t)strip * kStrip >= d.ku_ext) return false;
    const uint32_t left = d.ku_ext - strip * kStrip;
    const int V = d.unit_bytes;
    for (uint32_t u = 0; u < (uint32_t)kStrip && u < left; ++u) {
      bool load = d.input >= 0, live = true;
      for (int c = 0; c < nc; ++c) {
        const int64_t v = acc[c] + d.cons[c].off + (int64_t)u * d.ku_coef[c];
        if (v > INT32_MAX || v < INT32_MIN) return false;
        const bool ok = (uint32_t)(int32_t)v < (uint32_t)d.cons[c].extent;
        if (c < d.n_guards) load = load && ok; else live = live && ok;
      }
      if (!live) continue;
      const int64_t oo = o + (int64_t)u * d.ku_ds, sso = s + (int64_t)u * d.ku_ss;
      if (oo % V || oo < 0 || oo + V > out_bytes) return false;
      if (load && (sso % V || sso < 0 || sso + V > in_bytes)) return false;
    }
    return true;
  }
  bool load = d.input >= 0, live = true;
  for (int c = 0; c < nc; ++c) {
    const int64_t v = acc[c] + d.cons[c].off;
    if (v > INT32_MAX || v < INT32_MIN) return false;
    const bool ok = (uint32_t)(int32_t)v < (uint32_t)d.cons[c].extent;
    if (c < d.n_guards) load = load && ok; else live = live && ok;
  }
  if (!live) return true;
  const int V = d.unit_bytes;
  if (o % V || o < 0 || o + V > out_bytes) return false;
  if (load && (s % V || s < 0 || s + V > in_bytes)) return false;
  return true;
}

static bool check_affine_piece(const DevPiece &d, int64_t in_bytes, int64_t out_bytes) {
  if (d.n_items == 0) return true;
  if (d.n_items <= (1u << 18)) {
    for (uint64_t L = 0; L < d.n_items; ++L)
      if (!check_affine_item(d, L, in_bytes, out_bytes)) return false;
    return true;
  }
  uint64_t x = 0x9E3779B97F4A7C15ull;
  for (int t = 0; t < (1 << 16); ++t) {
    x ^= x << 13; x ^= x >> 7; x ^= x << 17;  // xorshift64
    uint64_t L = (t == 0) ? 0 : (t == 1) ? d.n_items - 1 : x % d.n_items;
    if (!check_affine_item(d, L, in_bytes, out_bytes)) return false;
  }
  // the far corner of every loop on its own
  uint64_t mult = 1;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    if (!check_affine_item(d, mult * (d.ext[k] - 1), in_bytes, out_bytes)) return false;
    mult *= d.ext[k];
  }
  return true;
}

// ---------------------------------------------------------------------------
// Transpose family.  A piece qualifies when its destination-contiguous loop is
// not its source-contiguous loop, it has no constraints, and all vector
// addresses are 16-byte aligned.  The a index (destination-contiguous) and the
// b index (source-contiguous) may each merge a second loop that is contiguous
// on that one side only (e.g. (h, w) is one run in an NCHW source but two
// strides in a padded NHWC destination).
// ---------------------------------------------------------------------------
// Tile counts of a transpose descriptor whose extents and batch loops are set: tiles of `ca` 16-byte chunks of a
// by up to kTileB * 8 / ca elements of b (1024 chunks either way).  With `even` the step along b is shortened to the smallest multiple of
// a chunk that still covers ext_b with the same number of tiles, so that no tile is left nearly empty
// (784 = 7 x 112 instead of 6 x 128 + 16).
static bool set_transpose_tiles(DevPiece *d, int ca, bool even) {
  const int es = d->unit_bytes, epu = 16 / es;
  const uint32_t ta = (uint32_t)(ca * epu), tb = (uint32_t)(kTileB * 8 / ca);
  d->tile_ca = ca;
  d->tiles_a = (d->ext_a + ta - 1) / ta;
  d->tiles_b = (d->ext_b + tb - 1) / tb;
  d->step_b = tb;
  if (even) {
    const uint32_t per = (d->ext_b + d->tiles_b - 1) / d->tiles_b;
    d->step_b = std::min(tb, (per + epu - 1) / epu * epu);
  }
  d->fd_tiles_a = make_fastdiv(d->tiles_a);
  d->fd_tiles_b = make_fastdiv(d->tiles_b);
  unsigned __int128 blocks = (unsigned __int128)d->tiles_a * d->tiles_b;
  for (int j = 0; j < d->n_loops; ++j) blocks *= d->ext[j];
  if (blocks > 0x7FFFFFFFull) return false;
  d->n_blocks = (uint32_t)blocks;
  d->n_items = (uint64_t)blocks;
  return true;
}

// The flat-destination kernel for a transpose descriptor built with single elements as units: b is one loop whose
// rows follow each other in the destination, every source access is an aligned 16-byte chunk along b, and every
// panel (all of a by step_b of b) starts on a 16-byte boundary of the destination.  Chooses step_b and the lanes
// per a; returns false when the piece does not qualify.
constexpr int kFlatMaxPanelBytes = 100 * 1024;  // two blocks per SM
static bool set_flat_panels(DevPiece *d) {
  const int es = d->unit_bytes, epu = 16 / es;
  if (d->fd_b_in.d < d->ext_b || d->db[0] != (int64_t)d->ext_a * es || d->ext_b % epu) return false;
  if (d->soff % 16 || d->sa[0] % 16 || d->sa[1] % 16 || d->doff % 16) return false;
  for (int j = 0; j < d->n_loops; ++j)
    if (d->sstride[j] % 16 || d->dstride[j] % 16) return false;
  const uint64_t row_bytes = (uint64_t)d->ext_a * es;
  if (row_bytes * epu > (uint64_t)kFlatMaxPanelBytes) return false;
  // step_b: 16/es elements times a power of two.  Measured on 2-byte elements: panels near 12-24 KB run best (eight
  // blocks of 256 threads per SM), but 64 bytes of b per a are worth a larger panel (rows of 1.4-2.4 KB: 47-78 KB
  // panels, two or four blocks of 512 threads per SM); with 32 bytes of b the shifted kernel is as fast or faster.
  const uint32_t min_bt = 64u / es, max_bt = 256u / es;
  if (row_bytes * min_bt > (uint64_t)kFlatMaxPanelBytes || d->ext_b < min_bt) return false;
  uint32_t bt = min_bt;
  int lg = 2;
  while (bt * 2 <= max_bt && bt * 2 <= d->ext_b && row_bytes * bt * 2 <= 24u * 1024u) {
    bt *= 2;
    ++lg;
  }
  d->tr_unit = -2;
  d->tile_ca = lg;
  d->step_b = bt;
  d->tiles_a = 1;
  d->tiles_b = (d->ext_b + bt - 1) / bt;
  d->fd_tiles_a = make_fastdiv(1);
  d->fd_tiles_b = make_fastdiv(d->tiles_b);
  unsigned __int128 blocks = d->tiles_b;
  for (int j = 0; j < d->n_loops; ++j) blocks *= d->ext[j];
  if (blocks > 0x7FFFFFFFull) return false;
  // a handful of large panels would leave most SMs idle: the tiled kernels cut such a piece finer
  if (row_bytes * bt > 24u * 1024u && blocks < (unsigned __int128)kDefaultSms) return false;
  d->n_blocks = (uint32_t)blocks;
  d->n_items = (uint64_t)blocks;
  return true;
}
// The mirror image for the flat-source kernel (tr_unit = -3): a is one loop whose rows follow each other in the
// SOURCE, every destination access is an aligned 16-byte chunk along a; step_b holds the elements of a per panel.
static bool set_flat_source_panels(DevPiece *d) {
  const int es = d->unit_bytes, epu = 16 / es;
  if (d->fd_a_in.d < d->ext_a || d->sa[0] != (int64_t)d->ext_b * es || d->ext_a % epu) return false;
  if (d->doff % 16 || d->db[0] % 16 || d->db[1] % 16 || d->soff % 16) return false;
  for (int j = 0; j < d->n_loops; ++j)
    if (d->sstride[j] % 16 || d->dstride[j] % 16) return false;
  const uint64_t row_bytes = (uint64_t)d->ext_b * es;
  const uint32_t min_at = 64u / es, max_at = 256u / es;
  if (row_bytes * min_at > (uint64_t)kFlatMaxPanelBytes || d->ext_a < min_at) return false;
  uint32_t at = min_at;
  int lg = 2;
  while (at * 2 <= max_at && at * 2 <= d->ext_a && row_bytes * at * 2 <= 24u * 1024u) {
    at *= 2;
    ++lg;
  }
  d->tr_unit = -3;
  d->tile_ca = lg;
  d->step_b = at;
  d->tiles_b = 1;
  d->tiles_a = (d->ext_a + at - 1) / at;
  d->fd_tiles_b = make_fastdiv(1);
  d->fd_tiles_a = make_fastdiv(d->tiles_a);
  unsigned __int128 blocks = d->tiles_a;
  for (int j = 0; j < d->n_loops; ++j) blocks *= d->ext[j];
  if (blocks > 0x7FFFFFFFull) return false;
  if (row_bytes * at > 24u * 1024u && blocks < (unsigned __int128)kDefaultSms) return false;
  d->n_blocks = (uint32_t)blocks;
  d->n_items = (uint64_t)blocks;
  return true;
}
// bytes of a panel of either flat kernel: step_b elements of the panelled index by all of the other
static int flat_panel_bytes(const DevPiece &d) {
  return (int)((uint64_t)d.step_b * (d.tr_unit == -3 ? d.ext_b : d.ext_a) * d.unit_bytes);
}
static int flat_threads(int panel_bytes) { return panel_bytes > 24 * 1024 ? 512 : 256; }
// blocks of a flat kernel resident per SM: eight of 256 threads or two of 512 (registers), as far as 227 KB of shared
// memory hold their panels (1 KB per block is the system's)
static int flat_blocks_per_sm(int panel_bytes) {
  return std::max(1, std::min(flat_threads(panel_bytes) == 256 ? 8 : 2, 227 * 1024 / (panel_bytes + 1024)));
}

// the flat-destination kernel's address arithmetic for one block, replayed on the host
static bool check_flat_block(const DevPiece &d, uint32_t blk, int threads, int64_t in_bytes, int64_t out_bytes) {
  const int es = d.unit_bytes, epu = 16 / es;
  if ((es != 2 && es != 4) || d.step_b == 0 || d.step_b % epu || d.ext_b % epu || d.tiles_b == 0 || d.tile_ca < 0 ||
      d.tile_ca > 5 || ((uint32_t)epu << d.tile_ca) < d.step_b || (threads != 256 && threads != 512) ||
      (uint64_t)d.tiles_b * d.step_b < d.ext_b || flat_panel_bytes(d) > kFlatMaxPanelBytes)
    return false;
  uint32_t t = blk;
  uint32_t q = host_fast_div(t, d.fd_tiles_b);
  if (q != t / d.tiles_b) return false;
  const uint32_t b0 = (t - q * d.tiles_b) * d.step_b;
  t = q;
  int64_t sbase = d.soff, dbase = d.doff;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    q = host_fast_div(t, d.fd[k]);
    if (q != t / d.ext[k]) return false;
    const uint32_t i = t - q * d.ext[k];
    t = q;
    sbase += (int64_t)i * d.sstride[k];
    dbase += (int64_t)i * d.dstride[k];
  }
  if (t != 0 || b0 >= d.ext_b) return false;
  const uint32_t nb = std::min<uint32_t>(d.step_b, d.ext_b - b0);
  const int64_t row_bytes = (int64_t)d.ext_a * es, panel = (int64_t)nb * row_bytes;
  // phase 2: the panel is one aligned range of the destination, a whole number of 16-byte units
  const int64_t D0 = dbase + (int64_t)b0 * d.db[0];
  if (d.db[0] != row_bytes || D0 % 16 || panel % 16 || D0 < 0 || D0 + panel > out_bytes) return false;
  // phase 1: every lane's loads and the elements it scatters
  const uint32_t lanes = 1u << d.tile_ca;
  for (uint32_t a = 0; a < d.ext_a; ++a) {
    const uint32_t a_hi = host_fast_div(a, d.fd_a_in);
    if (a_hi != a / d.fd_a_in.d) return false;
    const int64_t off = d.fd_a_in.d < d.ext_a ? (int64_t)(a - a_hi * d.fd_a_in.d) * d.sa[0] + (int64_t)a_hi * d.sa[1]
                                               : (int64_t)a * d.sa[0];
    for (uint32_t cb = 0; cb < lanes && cb * epu < nb; ++cb) {
      const int64_t g = sbase + (int64_t)b0 * es + (int64_t)cb * 16 + off;
      if (g % 16 || g < 0 || g + 16 > in_bytes) return false;
      const int64_t last = ((int64_t)cb * epu + epu - 1) * row_bytes + (int64_t)a * es;  // the lane's last element
      if (last + es > panel) return false;
    }
  }
  return true;
}

// the flat-source kernel's address arithmetic for one block, replayed on the host
static bool check_flat_source_block(const DevPiece &d, uint32_t blk, int threads, int64_t in_bytes, int64_t out_bytes) {
  const int es = d.unit_bytes, epu = 16 / es;
  if ((es != 2 && es != 4) || d.step_b == 0 || d.step_b % epu || d.ext_a % epu || d.tiles_a == 0 || d.tile_ca < 0 ||
      d.tile_ca > 5 || ((uint32_t)epu << d.tile_ca) < d.step_b || (threads != 256 && threads != 512) ||
      (uint64_t)d.tiles_a * d.step_b < d.ext_a || flat_panel_bytes(d) > kFlatMaxPanelBytes)
    return false;
  uint32_t t = blk;
  uint32_t q = host_fast_div(t, d.fd_tiles_a);
  if (q != t / d.tiles_a) return false;
  const uint32_t a0 = (t - q * d.tiles_a) * d.step_b;
  t = q;
  int64_t sbase = d.soff, dbase = d.doff;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    q = host_fast_div(t, d.fd[k]);
    if (q != t / d.ext[k]) return false;
    const uint32_t i = t - q * d.ext[k];
    t = q;
    sbase += (int64_t)i * d.sstride[k];
    dbase += (int64_t)i * d.dstride[k];
  }
  if (t != 0 || a0 >= d.ext_a) return false;
  const uint32_t na = std::min<uint32_t>(d.step_b, d.ext_a - a0);
  const int64_t row_bytes = (int64_t)d.ext_b * es, panel = (int64_t)na * row_bytes;
  // phase 1: the panel is one aligned range of the source, a whole number of 16-byte units
  const int64_t S0 = sbase + (int64_t)a0 * d.sa[0];
  if (d.sa[0] != row_bytes || S0 % 16 || panel % 16 || S0 < 0 || S0 + panel > in_bytes) return false;
  // phase 2: every lane's stores and the elements it gathers
  const uint32_t lanes = 1u << d.tile_ca;
  for (uint32_t b = 0; b < d.ext_b; ++b) {
    const uint32_t b_hi = host_fast_div(b, d.fd_b_in);
    if (b_hi != b / d.fd_b_in.d) return false;
    const int64_t off = d.fd_b_in.d < d.ext_b ? (int64_t)(b - b_hi * d.fd_b_in.d) * d.db[0] + (int64_t)b_hi * d.db[1]
                                               : (int64_t)b * d.db[0];
    for (uint32_t ca = 0; ca < lanes && ca * epu < na; ++ca) {
      const int64_t g = dbase + (int64_t)a0 * es + (int64_t)ca * 16 + off;
      if (g % 16 || g < 0 || g + 16 > out_bytes) return false;
      const int64_t last = ((int64_t)ca * epu + epu - 1) * row_bytes + (int64_t)b * es;  // the lane's last element
      if (last + es > panel) return false;
    }
  }
  return true;
}

// A 16-byte transpose piece whose extent along a leaves a remainder of at most half a tile is cut in two: whole
// tiles, and the remainder as a piece of its own on the narrow tile (64 bytes of a by 256 elements of b), which
// would otherwise travel in half-empty tiles.  Returns false when the piece stays as it is.
static bool split_a_remainder(const DevPiece &d, DevPiece *whole, DevPiece *rest) {
  const int es = d.unit_bytes, epu = 16 / es;
  const uint32_t ta = (uint32_t)(8 * epu);
  if (d.tr_unit != 16 || d.tile_ca != 8 || d.fd_a_in.d < d.ext_a) return false;  // a merges two loops: not cut
  const uint32_t rem = d.ext_a % ta;
  if (d.ext_a <= ta || rem == 0 || rem > ta / 2) return false;
  *whole = d;
  whole->ext_a = d.ext_a - rem;
  whole->fd_a_in = make_fastdiv(whole->ext_a);
  *rest = d;
  rest->ext_a = rem;
  rest->fd_a_in = make_fastdiv(rem);
  rest->soff = d.soff + (int64_t)whole->ext_a * d.sa[0];
  rest->doff = d.doff + (int64_t)whole->ext_a * es;
  return set_transpose_tiles(whole, 8, true) && set_transpose_tiles(rest, 4, true);
}

static bool build_transpose_piece(const Piece &p, int es, int ptr_align, int64_t in_bytes, DevPiece *d,
                                  bool allow_flat = true) {
  if (es > 8 || p.src == AMAP_CONST || p.qa.on || !p.guards.empty() || !p.domain.empty()) return false;
  const int n = p.n();
  if (n < 2) return false;
  const int ia = n - 1;
  if (p.dst.c[ia] != 1 || p.srcoff.c[ia] == 1) return false;
  int ib = -1;
  for (int k = 0; k < n - 1; ++k)
    if (p.srcoff.c[k] == 1) ib = k;
  if (ib < 0) return false;
  // second loop of a: next in destination order, contiguous with ia on the destination side
  int ia_hi = -1;
  if (ia - 1 >= 0 && ia - 1 != ib && p.dst.c[ia - 1] == p.ext[ia]) ia_hi = ia - 1;
  // second loop of b: contiguous with ib on the source side
  int ib_hi = -1;
  for (int k = 0; k < n; ++k)
    if (k != ia && k != ia_hi && k != ib && p.srcoff.c[k] == p.ext[ib]) ib_hi = k;
  auto try_build = [&](int a_hi, int b_hi, int ub) -> bool {
    const int epu = ub / es;
    const int64_t ext_a = p.ext[ia] * (a_hi >= 0 ? p.ext[a_hi] : 1);
    const int64_t ext_b = p.ext[ib] * (b_hi >= 0 ? p.ext[b_hi] : 1);
    if (ext_a % epu || ext_b % epu || ext_a > INT32_MAX || ext_b > INT32_MAX) return false;
    memset(d, 0, sizeof *d);
    d->kind = kDevTranspose;
    d->input = p.src;
    d->out = p.out;
    d->unit_bytes = es;
    d->tr_unit = ub;
    d->soff = p.srcoff.c0 * es;
    d->doff = p.dst.c0 * es;
    d->ext_a = (uint32_t)ext_a;
    d->ext_b = (uint32_t)ext_b;
    d->fd_a_in = make_fastdiv((uint32_t)p.ext[ia]);
    d->fd_b_in = make_fastdiv((uint32_t)p.ext[ib]);
    d->sa[0] = p.srcoff.c[ia] * es;
    d->sa[1] = a_hi >= 0 ? p.srcoff.c[a_hi] * es : 0;
    d->db[0] = p.dst.c[ib] * es;
    d->db[1] = b_hi >= 0 ? p.dst.c[b_hi] * es : 0;
    bool aligned = (d->soff % ub == 0) && (d->doff % ub == 0) && (d->sa[0] % ub == 0) && (d->sa[1] % ub == 0) &&
                   (d->db[0] % ub == 0) && (d->db[1] % ub == 0);
    int j = 0;
    for (int k = 0; k < n; ++k) {
      if (k == ia || k == a_hi || k == ib || k == b_hi) continue;
      if (j >= kDevMaxLoops) return false;
      d->ext[j] = (uint32_t)p.ext[k];
      d->fd[j] = make_fastdiv((uint32_t)p.ext[k]);
      d->sstride[j] = p.srcoff.c[k] * es;
      d->dstride[j] = p.dst.c[k] * es;
      if (d->sstride[j] % ub || d->dstride[j] % ub) aligned = false;
      ++j;
    }
    if (!aligned) return false;
    d->n_loops = j;
    // the 16-byte kernel has tile shapes for pieces that are short in a (4 chunks of a by 256 elements of b) or in
    // b (16 chunks by 64 elements, 32 chunks by 32 elements; their rows must stay 128 bytes long)
    int ca = 8;
    if (ub == 16) {
      if (ext_a <= 4 * (16 / es)) ca = 4;
      else if (ext_b <= 32 && es >= 4) ca = 32;
      else if (ext_b <= 64 && es >= 2) ca = 16;
    }
    return set_transpose_tiles(d, ca, ub == 16);
  };
  // Accesses of `ub` bytes on both sides.  Units of a single element gain nothing over the strip kernel's gather
  // (measured): at least two per access.
  auto try_unit = [&](int ub) -> bool {
    if (ub > ptr_align || ub < 2 * es) return false;
    if (try_build(ia_hi, ib_hi, ub)) return true;
    if (ib_hi >= 0 && try_build(ia_hi, -1, ub)) return true;
    if (ia_hi >= 0 && try_build(-1, ib_hi, ub)) return true;
    if (ia_hi >= 0 && ib_hi >= 0 && try_build(-1, -1, ub)) return true;
    return false;
  };
  // Order of preference, as measured on 2-byte elements (TB/s): 16-byte units on both sides 6.5; rows that follow
  // each other on the misaligned side and are short enough for a panel: the flat kernels 4.4-5.3; otherwise the
  // realigning kernel 4.0-5.0 for a misaligned source, 8-byte units 3.4-4.4 or the shifted-destination kernel
  // 3.2-4.2 for a misaligned destination; 4-byte units 2.9.
  if (try_unit(16)) return true;
  // source rows that follow each other in memory, destination rows aligned: the flat-source kernel (tr_unit = -3),
  // whatever the alignment of the source rows
  if (allow_flat && (es == 2 || es == 4) && ptr_align >= 16 && try_build(-1, ib_hi, es) &&
      set_flat_source_panels(d))
    return true;
  // source rows misaligned, destination rows aligned: the realigning kernel (tr_unit = -1; tile 8 x 14 chunks)
  if (es <= 4 && ptr_align >= 16 && try_build(ia_hi, ib_hi, es) && d->ext_a % (16 / es) == 0 && d->doff % 16 == 0 &&
      d->db[0] % 16 == 0 && d->db[1] % 16 == 0) {
    bool dst_aligned = true;
    for (int j = 0; j < d->n_loops; ++j) dst_aligned = dst_aligned && d->dstride[j] % 16 == 0;
    if (dst_aligned) {
      const int epu16 = 16 / es;
      d->tr_unit = -1;
      d->src_bytes = in_bytes;
      d->tiles_a = (d->ext_a + 8 * epu16 - 1) / (8 * epu16);
      d->tiles_b = (d->ext_b + 14 * epu16 - 1) / (14 * epu16);
      d->fd_tiles_a = make_fastdiv(d->tiles_a);
      d->fd_tiles_b = make_fastdiv(d->tiles_b);
      unsigned __int128 blocks = (unsigned __int128)d->tiles_a * d->tiles_b;
      for (int j = 0; j < d->n_loops; ++j) blocks *= d->ext[j];
      if (blocks <= 0x7FFFFFFFull) {
        d->n_blocks = (uint32_t)blocks;
        d->n_items = (uint64_t)blocks;
        return true;
      }
    }
  }
  // destination rows that follow each other in memory, source rows aligned: the flat-destination kernel
  // (tr_unit = -2), whatever the alignment of the destination rows
  if (allow_flat && (es == 2 || es == 4) && ptr_align >= 16 && try_build(ia_hi, -1, es) &&
      set_flat_panels(d))
    return true;
  if (try_unit(8)) return true;
  // destination rows misaligned, source rows aligned: the shifted-destination kernel (tr_unit = 0; it stores whole
  // slots of the destination's own 16-byte grid; rows at least one slot long, so that a slot spans two rows at most)
  if (es <= 4 && ptr_align >= 16 && try_build(ia_hi, ib_hi, es) && d->ext_b % (16 / es) == 0 && d->soff % 16 == 0 &&
      d->sa[0] % 16 == 0 && d->sa[1] % 16 == 0 && d->ext_a >= (uint32_t)(16 / es)) {
    bool src_aligned = true;
    for (int j = 0; j < d->n_loops; ++j) src_aligned = src_aligned && d->sstride[j] % 16 == 0;
    if (src_aligned) {
      d->tr_unit = 0;
      d->src_bytes = in_bytes;
      // row b + 1 follows row b in memory (b is one loop whose destination stride is the row's length)
      d->shift_wrap = (d->fd_b_in.d >= d->ext_b && d->db[0] == (int64_t)d->ext_a * es) ? 1 : 0;
      return true;  // tiles and blocks as try_build computed them: slot starts in 8 chunks of a by kTileB of b
    }
  }
  if (try_unit(4)) return true;
  if (try_unit(2)) return true;
  return false;
}

// the shifted-destination kernel's address arithmetic for one block, replayed on the host
static bool check_shifted_block(const DevPiece &d, uint32_t blk, int64_t in_bytes, int64_t out_bytes) {
  const int es = d.unit_bytes, epu = 16 / es, ta = 8 * epu;
  if (d.ext_b % epu || d.ext_a < (uint32_t)epu) return false;
  uint32_t t = blk;
  uint32_t q = t / d.tiles_b;
  const uint32_t b0 = (t - q * d.tiles_b) * kTileB;
  t = q;
  q = t / d.tiles_a;
  const uint32_t a0 = (t - q * d.tiles_a) * ta;
  t = q;
  int64_t sbase = d.soff, dbase = d.doff;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    q = t / d.ext[k];
    sbase += (int64_t)(t - q * d.ext[k]) * d.sstride[k];
    dbase += (int64_t)(t - q * d.ext[k]) * d.dstride[k];
    t = q;
  }
  if (t != 0 || a0 >= d.ext_a || b0 >= d.ext_b) return false;
  const uint32_t end_b = std::min<uint32_t>(b0 + kTileB, d.ext_b);
  const bool holds_row_end = a0 + ta + epu > d.ext_a, rows_follow = d.shift_wrap != 0;
  auto src_ok = [&](uint32_t a, uint32_t b) {  // an aligned 16-byte load of the source
    const uint32_t a_hi = a / d.fd_a_in.d;
    const int64_t s = sbase + (int64_t)(a - a_hi * d.fd_a_in.d) * d.sa[0] + (int64_t)a_hi * d.sa[1] + (int64_t)b * es;
    return s % 16 == 0 && s >= 0 && s + 16 <= in_bytes;
  };
  for (int r = 0; r < ta + 2 * epu; ++r) {
    const uint32_t a = r < ta + epu ? a0 + r : (uint32_t)(r - (ta + epu));
    const bool wanted = r < ta + epu ? a < d.ext_a : (holds_row_end && rows_follow && a < d.ext_a);
    for (uint32_t b = b0; wanted && b < end_b; b += epu)
      if (!src_ok(a, b)) return false;
  }
  auto row_start = [&](uint32_t b) {
    const uint32_t b_hi = b / d.fd_b_in.d;
    return dbase + (int64_t)(b - b_hi * d.fd_b_in.d) * d.db[0] + (int64_t)b_hi * d.db[1];
  };
  // the slots of a row are the same whether the kernel walks them row by row or, for short rows, along the flat range
  for (uint32_t b = b0; b < end_b; ++b) {
    const int64_t D = row_start(b);
    if (D < 0 || D % es || D + (int64_t)d.ext_a * es > out_bytes) return false;
    if (rows_follow && b + 1 < end_b && row_start(b + 1) != D + (int64_t)d.ext_a * es) return false;
    const uint32_t head = (uint32_t)((16 - (int)(D & 15)) & 15) / es;
    for (int k = 0; k < 8; ++k) {
      const uint32_t a_s = a0 + head + (uint32_t)k * epu;
      if (a_s >= d.ext_a) continue;
      const bool next_col = rows_follow && b + 1 < end_b;
      if (a_s + epu > d.ext_a && next_col && !holds_row_end) return false;  // would read wrap rows that were not loaded
      if (a_s + epu <= d.ext_a || next_col) {  // a whole slot: aligned and inside
        const int64_t A = D + (int64_t)a_s * es;
        if (A % 16 || A < 0 || A + 16 > out_bytes) return false;
      }
      if (a_s - a0 + epu > (uint32_t)(ta + epu)) return false;  // beyond the rows the tile holds
    }
  }
  return true;
}

// the realigning kernel's address arithmetic for one block, replayed on the host
static bool check_realign_block(const DevPiece &d, uint32_t blk, int64_t in_bytes, int64_t out_bytes) {
  const int es = d.unit_bytes, epu = 16 / es, ta = 8 * epu, tbr = 14 * epu;
  if (d.src_bytes != in_bytes || d.ext_a % epu) return false;
  uint32_t t = blk;
  uint32_t q = t / d.tiles_b;
  const uint32_t b0 = (t - q * d.tiles_b) * tbr;
  t = q;
  q = t / d.tiles_a;
  const uint32_t a0 = (t - q * d.tiles_a) * ta;
  t = q;
  int64_t sbase = d.soff, dbase = d.doff;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    q = t / d.ext[k];
    sbase += (int64_t)(t - q * d.ext[k]) * d.sstride[k];
    dbase += (int64_t)(t - q * d.ext[k]) * d.dstride[k];
    t = q;
  }
  if (t != 0 || a0 >= d.ext_a || b0 >= d.ext_b) return false;
  const int nb = (int)std::min<uint32_t>(tbr, d.ext_b - b0);
  for (uint32_t a = a0; a < std::min<uint32_t>(a0 + ta, d.ext_a); ++a) {
    const uint32_t a_hi = a / d.fd_a_in.d;
    const int64_t g = sbase + (int64_t)(a - a_hi * d.fd_a_in.d) * d.sa[0] + (int64_t)a_hi * d.sa[1] + (int64_t)b0 * es;
    if (g < 0 || g % es || g + (int64_t)nb * es > in_bytes) return false;
    // the row's bytes must be covered by at most 15 aligned chunks, so that lane 14 holds the last one needed
    if ((((g + (int64_t)nb * es + 15) & ~(int64_t)15) - (g & ~(int64_t)15)) / 16 > 15) return false;
    for (int b_l = 0; b_l < nb; ++b_l) {
      const uint32_t b = b0 + b_l, b_hi = b / d.fd_b_in.d;
      const int64_t o = dbase + (int64_t)(b - b_hi * d.fd_b_in.d) * d.db[0] + (int64_t)b_hi * d.db[1] + (int64_t)a * es;
      if (o < 0 || o + es > out_bytes || ((a - a0) % epu == 0 && o % 16)) return false;
    }
  }
  return true;
}

// the kernel's address arithmetic for one block, replayed on the host
static bool check_transpose_block(const DevPiece &d, uint32_t blk, int64_t in_bytes, int64_t out_bytes) {
  if (d.tr_unit == -2) return check_flat_block(d, blk, flat_threads(flat_panel_bytes(d)), in_bytes, out_bytes);
  if (d.tr_unit == -3) return check_flat_source_block(d, blk, flat_threads(flat_panel_bytes(d)), in_bytes, out_bytes);
  if (d.tr_unit == 0) return check_shifted_block(d, blk, in_bytes, out_bytes);
  if (d.tr_unit < 0) return check_realign_block(d, blk, in_bytes, out_bytes);
  const int es = d.unit_bytes, epu = 16 / es, ca = d.tile_ca, ta = ca * epu;
  const bool shape_ok = ca == 8 || (d.tr_unit == 16 && (ca == 4 || (ca == 16 && es >= 2) || (ca == 32 && es >= 4)));
  if (!shape_ok || d.step_b == 0 || d.step_b % epu || d.step_b > (uint32_t)(kTileB * 8 / ca) ||
      (uint64_t)d.tiles_b * d.step_b < d.ext_b || (uint64_t)d.tiles_a * ta < d.ext_a)
    return false;
  uint32_t t = blk;
  uint32_t q = host_fast_div(t, d.fd_tiles_b);
  if (q != t / d.tiles_b) return false;
  const uint32_t b0 = (t - q * d.tiles_b) * d.step_b;
  const uint32_t end_b = std::min<uint32_t>(d.ext_b, b0 + d.step_b);
  t = q;
  q = host_fast_div(t, d.fd_tiles_a);
  if (q != t / d.tiles_a) return false;
  const uint32_t a0 = (t - q * d.tiles_a) * ta;
  t = q;
  int64_t sbase = d.soff, dbase = d.doff;
  for (int k = d.n_loops - 1; k >= 0; --k) {
    q = host_fast_div(t, d.fd[k]);
    if (q != t / d.ext[k]) return false;
    const uint32_t i = t - q * d.ext[k];
    t = q;
    sbase += (int64_t)i * d.sstride[k];
    dbase += (int64_t)i * d.dstride[k];
  }
  if (t != 0) return false;
  const int ub = d.tr_unit, epn = ub / es, rb = kTileB * 8 / ca * es, cbu = rb / ub, nca = ta / epn;
  auto swizzle = [&](int chunk_a) { return ca >= 8 ? (chunk_a & 7) : chunk_a * (8 / ca); };
  auto tile_off = [&](int row, int col) { return row * rb + ((((col >> 4) ^ swizzle(row / epu)) << 4) | (col & 15)); };
  // phase 2 below visits the kernel's (chunk of a, b) pairs in plain order; the kernel deals the same pairs out to
  // its lanes in another order
  for (int idx = 0; idx < kTileBytes / ub; ++idx) {
    {  // phase 1
      const int a_l = idx / cbu, cu = idx % cbu;
      const uint32_t a = a0 + a_l, b = b0 + cu * epn;
      if (a < d.ext_a && b < end_b) {
        const uint32_t a_hi = host_fast_div(a, d.fd_a_in);
        if (a_hi != a / d.fd_a_in.d) return false;
        const uint32_t a_lo = a - a_hi * d.fd_a_in.d;
        const int64_t s = sbase + (int64_t)a_lo * d.sa[0] + (int64_t)a_hi * d.sa[1] + (int64_t)b * es;
        if (s % ub || s < 0 || s + ub > in_bytes) return false;
        const int sm = tile_off(a_l, cu * ub);
        if (sm < 0 || sm + ub > kTileBytes || sm % ub) return false;
      }
    }
    {  // phase 2
      const int ca = idx % nca, b_l = idx / nca;
      const uint32_t a = a0 + ca * epn, b = b0 + b_l;
      if (a < d.ext_a && b < end_b) {
        const uint32_t b_hi = host_fast_div(b, d.fd_b_in);
        if (b_hi != b / d.fd_b_in.d) return false;
        const uint32_t b_lo = b - b_hi * d.fd_b_in.d;
        const int64_t o = dbase + (int64_t)b_lo * d.db[0] + (int64_t)b_hi * d.db[1] + (int64_t)a * es;
        if (o % ub || o < 0 || o + ub > out_bytes) return false;
        const int sm = tile_off(ca * epn + epn - 1, b_l * es);
        if (sm < 0 || sm + es > kTileBytes) return false;
      }
    }
  }
  return true;
}

static bool check_transpose_piece(const DevPiece &d, int64_t in_bytes, int64_t out_bytes) {
  if (d.n_blocks <= 256) {
    for (uint32_t b = 0; b < d.n_blocks; ++b)
      if (!check_transpose_block(d, b, in_bytes, out_bytes)) return false;
    return true;
  }
  uint64_t x = 0x9E3779B97F4A7C15ull;
  for (int t = 0; t < 256; ++t) {
    x ^= x << 13; x ^= x >> 7; x ^= x << 17;  // xorshift64
    const uint32_t b = (t == 0) ? 0 : (t == 1) ? d.n_blocks - 1 : (uint32_t)(x % d.n_blocks);
    if (!check_transpose_block(d, b, in_bytes, out_bytes)) return false;
  }
  return true;
}

// ---------------------------------------------------------------------------
// Building the launches of one stage
// ---------------------------------------------------------------------------
struct PlanCtx {
  const Map &m;
  const amap_plan_opts &o;
  int es;
  const std::vector<int64_t> &slot_numel;  // elements behind each source slot: inputs, then temporaries
  const std::vector<int> &unit_of;         // unit width chosen per piece (affine / strip kernels)
  const std::vector<DevPiece> &tr;         // transpose descriptor per piece (valid where is_tr)
  const std::vector<char> &is_tr;
  std::vector<char> placed;                // piece already belongs to a launch
  amap_plan_t *pl;
};

// bytes of the tensor piece q writes: the stage's temporary, or the piece's own output in the final stage
static int64_t piece_out_bytes(const PlanCtx &c, int stage, size_t q) {
  const StageInfo &st = c.m.stages[stage];
  if (st.dst_temp >= 0 || c.m.out_numels.empty()) return st.numel * c.es;
  return c.m.out_numels[c.m.pieces[q].out] * c.es;
}

static int plan_fail(int rc, size_t piece) {
  if (log_enabled()) fprintf(stderr, "[amap] planning piece %zu failed (%d)\n", piece, rc);
  return rc;
}

static bool append_piece(amap_plan_t *pl, Launch *L, DevPiece d) {
  if ((uint64_t)L->n_blocks + d.n_blocks > 0x7FFFFFFFull) return false;
  d.first_block = L->n_blocks;
  L->n_blocks += d.n_blocks;
  L->n_pieces++;
  pl->table.push_back(d);
  return true;
}

// One launch of the transpose kernel per (access width, offset width) present.  Fill pieces with 16-byte units
// and no constraints ride in the 16-byte launch, so that padding borders do not cost a launch of their own; their
// blocks come last (measured: 0.4 us faster on a 69 MB padded transpose than with the fills first).
static int plan_stage_transposes(PlanCtx &c, int stage) {
  const StageInfo &st = c.m.stages[stage];
  const size_t q_lo = st.first_piece, q_hi = q_lo + st.n_pieces;
  for (int access : {16, 8, 4, 2, 0, -1, -2, -3})
    for (int wide = 0; wide < 2; ++wide) {
      Launch L{kDevTranspose, c.es, access, wide, (int)c.pl->table.size(), 0, 0, stage};
      std::vector<DevPiece> transposes, fills;
      std::vector<size_t> taken;
      for (size_t q = q_lo; q < q_hi; ++q) {
        if (!c.is_tr[q] || c.tr[q].tr_unit != access) continue;
        const DevPiece &d = c.tr[q];
        const int64_t in_bytes = c.slot_numel[d.input] * c.es, out_bytes = piece_out_bytes(c, stage, q);
        const bool needs_wide = (in_bytes >= (1ll << 32) || out_bytes >= (1ll << 32)) && access > 0;
        if ((int)needs_wide != wide) continue;
        if (!check_transpose_piece(d, in_bytes, out_bytes)) return plan_fail(AMAP_EOVERFLOW, q);
        DevPiece whole, rest;
        if (split_a_remainder(d, &whole, &rest) && check_transpose_piece(whole, in_bytes, out_bytes) &&
            check_transpose_piece(rest, in_bytes, out_bytes)) {
          transposes.push_back(whole);
          transposes.push_back(rest);
        } else {
          transposes.push_back(d);
        }
        taken.push_back(q);
      }
      if (transposes.empty()) continue;
      for (size_t q = q_lo; q < q_hi && access == 16; ++q) {
        const Piece &p = c.m.pieces[q];
        if (c.placed[q] || p.src != AMAP_CONST || c.unit_of[q] != 16 || !p.guards.empty() || !p.domain.empty()) continue;
        DevPiece d;
        if (build_affine_piece(p, c.es, 16, &d) != AMAP_OK || d.n_items == 0) continue;
        make_strip(&d);
        if (!check_affine_piece(d, 0, piece_out_bytes(c, stage, q))) return plan_fail(AMAP_EOVERFLOW, q);
        fills.push_back(d);
        taken.push_back(q);
      }
      for (const DevPiece &d : transposes)
        if (!append_piece(c.pl, &L, d)) return plan_fail(AMAP_EUNSUPPORTED, q_lo);
      for (const DevPiece &d : fills)
        if (!append_piece(c.pl, &L, d)) return plan_fail(AMAP_EUNSUPPORTED, q_lo);
      for (size_t q : taken) c.placed[q] = 1;
      if (access <= -2) {  // the block size and the shared memory of the largest panel serve the whole launch
        for (const DevPiece &d : transposes) L.smem = std::max(L.smem, flat_panel_bytes(d));
        L.threads = flat_threads(L.smem);
        L.paired = (access == -2 && c.es == 2) ? 1 : 0;
        for (const DevPiece &d : transposes)
          if (d.ext_a & 1u) L.paired = 0;
      }
      c.pl->launches.push_back(L);
    }
  return AMAP_OK;
}

// Everything else: one launch per (unit width, constraint slots, offset width, strip or per-unit kernel) present.
static int plan_stage_strips(PlanCtx &c, int stage) {
  const StageInfo &st = c.m.stages[stage];
  const size_t q_lo = st.first_piece, q_hi = q_lo + st.n_pieces;
  for (int V = 16; V >= 1; V >>= 1)
    for (int cons : {0, 2, kDevMaxCons})
      for (int wide = 0; wide < 2; ++wide)
        for (int kind : {(int)kDevStrip, (int)kDevAffine}) {
          Launch L{kind, V, cons, wide, (int)c.pl->table.size(), 0, 0, stage};
          for (size_t q = q_lo; q < q_hi; ++q) {
            if (c.placed[q] || c.unit_of[q] != V) continue;
            const Piece &p = c.m.pieces[q];
            const int n_cons = (int)(p.guards.size() + p.domain.size());
            if ((n_cons == 0 ? 0 : n_cons <= 2 ? 2 : kDevMaxCons) != cons) continue;
            const int64_t in_bytes = (p.src >= 0) ? c.slot_numel[p.src] * c.es : 0, out_bytes = piece_out_bytes(c, stage, q);
            if ((int)(in_bytes >= (1ll << 32) || out_bytes >= (1ll << 32)) != wide) continue;
            DevPiece d;
            const int rc = build_affine_piece(p, c.es, V, &d);
            if (rc != AMAP_OK) return plan_fail(rc, q);
            if (d.n_items == 0) {
              c.placed[q] = 1;
              continue;
            }
            if (c.o.force_kernel != AMAP_KERNEL_GATHER && d.qa_n == 0) make_strip(&d);
            if (d.kind != kind) continue;
            if (!check_affine_piece(d, in_bytes, out_bytes)) return plan_fail(AMAP_EOVERFLOW, q);
            if (!append_piece(c.pl, &L, d)) return plan_fail(AMAP_EUNSUPPORTED, q);
            c.placed[q] = 1;
          }
          if (L.n_pieces > 0) c.pl->launches.push_back(L);
        }
  return AMAP_OK;
}

// ---------------------------------------------------------------------------
// Batch slabs for amap_execute_host.  If the outermost loop of every piece is the same batch loop, advancing it
// moves every input and the output by one whole slab and nothing else of a piece leaves its slab, then slab k of
// the output needs only slab k of the inputs: the host entry point can upload, run and download slab by slab and
// overlap the three (PCIe is full duplex).  Guarded pieces are left alone (their unguarded offsets may point
// outside the slab).
// ---------------------------------------------------------------------------
static int plan_impl(const amap_map *map, int device, const amap_plan_opts *opts, bool allow_slabs, amap_plan_t **out_plan);
static cudaError_t allow_flat_panels();
static bool has_flat_launches(const amap_plan_t *plan);

static void plan_slabs(const Map &m, int device, const amap_plan_opts &o, amap_plan_t *pl) {
  if (m.stages.size() != 1 || m.pieces.empty() || m.out_numel == 0 || m.out_numels.size() > 1) return;
  const int64_t N = m.pieces[0].n() > 0 ? m.pieces[0].ext[0] : 0;
  if (N < 2 || m.out_numel % N) return;
  const int64_t DS = m.out_numel / N;
  for (int64_t n : m.in_numel)
    if (n % N) return;
  auto inside = [](const Aff &a, const std::vector<int64_t> &ext, int64_t slab) {
    Aff rest = a;
    rest.c[0] = 0;
    int64_t lo, hi;
    aff_range(rest, ext, &lo, &hi);
    return lo >= 0 && hi < slab;
  };
  for (const Piece &p : m.pieces) {
    if (p.n() < 1 || p.ext[0] != N || !p.guards.empty() || !p.domain.empty() || p.qa.on) return;
    if (p.dst.c[0] != DS || !inside(p.dst, p.ext, DS)) return;
    if (p.src != AMAP_CONST) {
      const int64_t SS = m.in_numel[p.src] / N;
      if (p.srcoff.c[0] != SS || !inside(p.srcoff, p.ext, SS)) return;
    }
  }
  int slabs = 1;
  for (int g = 2; g <= 8; ++g)
    if (N % g == 0) slabs = g;
  if (slabs < 2) return;
  const int64_t per = N / slabs;
  const int es = m.elem_size;
  amap_map sub;
  sub.m = m;
  sub.m.guard_views.clear();
  sub.m.domain_views.clear();
  for (Piece &p : sub.m.pieces) p.ext[0] = per;
  sub.m.out_numel = DS * per;
  sub.m.out_numels = {sub.m.out_numel};
  sub.m.stages[0].numel = sub.m.out_numel;
  for (size_t q = 0; q < m.in_numel.size(); ++q) sub.m.in_numel[q] = m.in_numel[q] / N * per;
  if ((sub.m.out_numel * es) % pl->pointer_align) return;
  for (int64_t n : sub.m.in_numel)
    if ((n * es) % pl->pointer_align) return;
  amap_plan_t *sp = nullptr;
  if (plan_impl(&sub, device, &o, false, &sp) != AMAP_OK) return;
  pl->slab_plan = sp;
  pl->n_slabs = slabs;
  pl->slab_out_bytes = sub.m.out_numel * es;
  for (int64_t n : sub.m.in_numel) pl->slab_in_bytes.push_back(n * es);
}

static int plan_impl(const amap_map *map, int device, const amap_plan_opts *opts, bool allow_slabs, amap_plan_t **out_plan) {
  if (!map || !out_plan) return AMAP_EINVAL;
  amap_plan_opts o;
  memset(&o, 0, sizeof o);
  if (opts) o = *opts;
  for (int r : o.reserved)
    if (r != 0) return AMAP_EINVAL;
  if (o.flags & ~(AMAP_PLAN_NO_PDL | AMAP_PLAN_NO_PREFETCH)) return AMAP_EINVAL;
  if (o.force_kernel < AMAP_KERNEL_AUTO || o.force_kernel > AMAP_KERNEL_FILL) return AMAP_EINVAL;
  const Map &m = map->m;
  const int es = m.elem_size;
  int align = o.pointer_align ? o.pointer_align : es;
  if (align < es || (align & (align - 1))) return AMAP_EINVAL;
  if ((int)(m.in_numel.size() + m.temp_numel.size()) > kMaxInputs) return AMAP_EUNSUPPORTED;
  std::vector<int64_t> slot_numel = m.in_numel;  // what a piece's source slot holds: inputs, then temporaries
  slot_numel.insert(slot_numel.end(), m.temp_numel.begin(), m.temp_numel.end());

  if (device < -1) return AMAP_EINVAL;
  if (device >= 0) {
    int n_dev = 0;
    CUDA_TRY(cudaGetDeviceCount(&n_dev));
    if (device >= n_dev) return AMAP_EINVAL;
  }

  amap_plan_t *pl = new (std::nothrow) amap_plan_t();
  if (!pl) return AMAP_ENOMEM;
  pl->device = device;
  pl->elem_size = es;
  pl->pointer_align = align;
  pl->pdl = !(o.flags & AMAP_PLAN_NO_PDL);
  pl->in_numel = m.in_numel;
  pl->in_used.assign(m.in_numel.size(), 0);
  for (const Piece &p : m.pieces)
    if (p.src >= 0 && p.src < (int)m.in_numel.size()) pl->in_used[p.src] = 1;
  pl->out_numel = m.out_numel;
  pl->out_numels = m.out_numels.empty() ? std::vector<int64_t>{m.out_numel} : m.out_numels;
  if ((int)pl->out_numels.size() > kMaxOutputs) {
    delete pl;
    return AMAP_EUNSUPPORTED;
  }
  pl->temp_numel = m.temp_numel;
  for (const StageInfo &st : m.stages) pl->stage_dst.push_back(st.dst_temp);
  memset(&pl->stats, 0, sizeof pl->stats);
  pl->stats.n_pieces = (int32_t)m.pieces.size();

  // Kernel family and unit width per piece
  std::vector<int> unit_of(m.pieces.size());
  std::vector<DevPiece> tr(m.pieces.size());
  std::vector<char> is_tr(m.pieces.size(), 0);
  std::vector<int64_t> reads(slot_numel.size(), 0);
  const bool allow_transpose = (o.force_kernel == AMAP_KERNEL_AUTO || o.force_kernel == AMAP_KERNEL_TRANSPOSE);
  for (size_t q = 0; q < m.pieces.size(); ++q) {
    const Piece &p = m.pieces[q];
    unit_of[q] = pick_unit(p, es, std::min(align, 16), o.force_kernel);
    int64_t pts = count_points(p);
    if (pts < 0) pts = 0;
    pl->stats.bytes_written += pts * es;
    int kind;
    if (p.src == AMAP_CONST) {
      pl->stats.bytes_filled += pts * es;
      kind = AMAP_KERNEL_FILL;
    } else {
      reads[p.src] += piece_unique_reads(p, slot_numel[p.src]);
      const bool contiguous = p.n() > 0 && p.dst.c[p.n() - 1] == 1 &&
                              (p.qa.on ? unit_of[q] > es : p.srcoff.c[p.n() - 1] == 1);
      if (!contiguous && allow_transpose && build_transpose_piece(p, es, align, slot_numel[p.src] * es, &tr[q])) {
        is_tr[q] = 1;
        kind = AMAP_KERNEL_TRANSPOSE;
      } else {
        kind = (unit_of[q] > es || contiguous) ? AMAP_KERNEL_COPY : AMAP_KERNEL_GATHER;
      }
    }
    pl->piece_kernel.push_back(kind);
  }
  for (size_t q = 0; q < reads.size(); ++q) pl->stats.bytes_read += std::min(reads[q], slot_numel[q]) * es;
  // A stage whose transposes would split between a flat kernel and the tiled kernel for the same misaligned side
  // (operands of a concat with enough channels for a panel and others with too few) runs them all on the tiled
  // kernel: one launch instead of two.
  for (const StageInfo &st : m.stages) {
    bool flat_src = false, realign = false, flat_dst = false, other_dst = false;
    for (size_t q = st.first_piece; q < (size_t)(st.first_piece + st.n_pieces); ++q) {
      if (!is_tr[q]) continue;
      flat_src = flat_src || tr[q].tr_unit == -3;
      realign = realign || tr[q].tr_unit == -1;
      flat_dst = flat_dst || tr[q].tr_unit == -2;
      other_dst = other_dst || tr[q].tr_unit == 0 || (tr[q].tr_unit > 0 && tr[q].tr_unit < 16);
    }
    for (size_t q = st.first_piece; q < (size_t)(st.first_piece + st.n_pieces); ++q) {
      if (!is_tr[q]) continue;
      if ((tr[q].tr_unit == -3 && realign) || (tr[q].tr_unit == -2 && other_dst)) {
        DevPiece d;
        const Piece &p = m.pieces[q];
        if (build_transpose_piece(p, es, align, slot_numel[p.src] * es, &d, false)) tr[q] = d;
      }
    }
  }

  PlanCtx ctx{m, o, es, slot_numel, unit_of, tr, is_tr, std::vector<char>(m.pieces.size(), 0), pl};
  for (int stage = 0; stage < (int)m.stages.size(); ++stage) {
    int rc = plan_stage_transposes(ctx, stage);
    if (rc == AMAP_OK) rc = plan_stage_strips(ctx, stage);
    if (rc != AMAP_OK) {
      delete pl;
      return rc;
    }
  }
  for (int k : pl->piece_kernel) {
    const int slot = (k == AMAP_KERNEL_GATHER) ? 0 : (k == AMAP_KERNEL_COPY) ? 1 : (k == AMAP_KERNEL_TRANSPOSE) ? 2 : 3;
    pl->stats.kernel_kind[slot]++;
  }
  pl->stats.n_launches = (int32_t)pl->launches.size();
  pl->stats.n_descriptors = (int32_t)pl->table.size();
  pl->stats.n_stages = (int32_t)m.stages.size();
  {
    // prefetch distance for the transpose kernel: the number of blocks resident at once (8 per SM).  A dry plan
    // knows no device: it assumes kDefaultSms, and amap_execute_static rescales the distances for the device it
    // runs on.
    int sms = kDefaultSms;
    if (device >= 0 && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) sms = kDefaultSms;
    const char *dist = getenv("AMAP_PREFETCH_DISTANCE");
    const int ahead = dist ? atoi(dist) : 8 * sms;
    for (DevPiece &d : pl->table)
      d.prefetch = (o.flags & AMAP_PLAN_NO_PREFETCH) ? 0 : (d.kind == kDevTranspose && ahead > 1) ? ahead : 1;
    // the flat kernels: as many blocks ahead as are resident with their block size and panel
    for (DevPiece &d : pl->table)
      if (d.kind == kDevTranspose && d.tr_unit <= -2 && d.prefetch > 1 && !dist)
        d.prefetch = sms * flat_blocks_per_sm(flat_panel_bytes(d));
    // plain copies (one loop of 16-byte units): the affine kernel looks one resident wave ahead too, up to 128 MB
    // (measured: 15.8 -> 15.1 us on 49 MB, 30.6 -> 30.2 us on 98 MB, but 154 -> 160 us on 512 MB)
    const uint64_t kCopyAheadMaxBytes = 128ull << 20;
    const char *cdist = getenv("AMAP_COPY_PREFETCH_DISTANCE");
    const int copy_ahead = cdist ? atoi(cdist) : 5 * sms;
    for (DevPiece &d : pl->table)
      if (d.kind == kDevAffine && d.n_loops == 1 && d.unit_bytes == 16 && d.prefetch == 1 && copy_ahead > 1 &&
          d.n_items * 16 <= kCopyAheadMaxBytes)
        d.prefetch = copy_ahead;
  }
  for (const Launch &L : pl->launches) {
    LaunchDesc ld;
    memset(&ld, 0, sizeof ld);
    if (L.n_pieces <= kParamPieces) {
      ld.n_pieces = L.n_pieces;
      for (int q = 0; q < L.n_pieces; ++q) ld.piece[q] = pl->table[L.first_piece + q];
    }
    pl->launch_desc.push_back(ld);
  }

  if (device < 0) {  // a dry plan: can be inspected, not executed
    *out_plan = pl;
    return AMAP_OK;
  }
  int prev = 0;
  cudaError_t e = cudaGetDevice(&prev);
  if (e == cudaSuccess) e = cudaSetDevice(device);
  if (e == cudaSuccess && !pl->table.empty()) {
    e = cudaMalloc((void **)&pl->dev_table, pl->table.size() * sizeof(DevPiece));
    if (e == cudaSuccess)
      e = cudaMemcpy(pl->dev_table, pl->table.data(), pl->table.size() * sizeof(DevPiece), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess && has_flat_launches(pl)) e = allow_flat_panels();
  pl->temps.assign(pl->temp_numel.size(), nullptr);
  for (size_t k = 0; k < pl->temps.size() && e == cudaSuccess; ++k)
    if (pl->temp_numel[k] > 0) e = cudaMalloc(&pl->temps[k], (size_t)pl->temp_numel[k] * es);
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    const int rc = cuda_fail(e, "amap_plan: device allocation");
    amap_plan_destroy(pl);
    return rc;
  }
  if (allow_slabs) plan_slabs(m, device, o, pl);  // best effort: without it amap_execute_host copies in one piece
  *out_plan = pl;
  return AMAP_OK;
}

extern "C" int amap_plan(const amap_map *map, int device, const amap_plan_opts *opts, amap_plan_t **out_plan) {
  return plan_impl(map, device, opts, true, out_plan);
}

extern "C" void amap_plan_destroy(amap_plan_t *plan) {
  if (!plan) return;
  if (plan->device < 0) {
    delete plan;
    return;
  }
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(plan->device);
  if (plan->dev_table) cudaFree(plan->dev_table);
  for (void *p : plan->temps)
    if (p) cudaFree(p);
  for (void *p : plan->stage_in)
    if (p) cudaFree(p);
  if (plan->stage_out) cudaFree(plan->stage_out);
  if (plan->slab_plan) amap_plan_destroy(plan->slab_plan);
  if (plan->h2d_stream) cudaStreamDestroy(plan->h2d_stream);
  if (plan->d2h_stream) cudaStreamDestroy(plan->d2h_stream);
  for (cudaEvent_t ev : plan->events) cudaEventDestroy(ev);
  cudaSetDevice(prev);
  delete plan;
}

extern "C" int amap_plan_stats(const amap_plan_t *plan, amap_stats *out) {
  if (!plan || !out) return AMAP_EINVAL;
  *out = plan->stats;
  return AMAP_OK;
}

extern "C" int amap_plan_launch_info(const amap_plan_t *plan, int32_t k, amap_launch_info *out) {
  if (!plan || !out || k < 0 || k >= (int32_t)plan->launches.size()) return AMAP_EINVAL;
  const Launch &L = plan->launches[k];
  memset(out, 0, sizeof *out);
  if (L.kind == kDevTranspose) {
    out->kernel = L.cons == -3 ? AMAP_LAUNCH_TRANSPOSE_FLAT_SOURCE : L.cons == -2 ? AMAP_LAUNCH_TRANSPOSE_FLAT : L.cons == -1 ? AMAP_LAUNCH_TRANSPOSE_REALIGN
                : L.cons == 0 ? AMAP_LAUNCH_TRANSPOSE_SHIFTED : AMAP_LAUNCH_TRANSPOSE;
    out->access = L.cons > 0 ? L.cons : 16;
    out->threads = L.threads ? L.threads : kTransposeThreads;
  } else {
    out->kernel = L.kind == kDevStrip ? AMAP_LAUNCH_STRIP : AMAP_LAUNCH_AFFINE;
    out->access = L.unit;
    out->threads = kAffineThreads;
  }
  out->n_descriptors = L.n_pieces;
  out->stage = L.stage;
  out->n_blocks = L.n_blocks;
  out->smem_bytes = L.smem;
  out->wide_offsets = L.wide;
  return AMAP_OK;
}

extern "C" int amap_plan_piece_kernel(const amap_plan_t *plan, int32_t k, int32_t *kind) {
  if (!plan || !kind || k < 0 || k >= (int32_t)plan->piece_kernel.size()) return AMAP_EINVAL;
  *kind = plan->piece_kernel[k];
  return AMAP_OK;
}

// One kernel launch.  With `pdl` the launch carries the programmatic-stream-serialisation attribute: the grid may
// become resident while the kernel before it on the stream drains; the kernels wait (griddepcontrol.wait) for that
// kernel's completion before they touch a caller buffer.
template <typename... P, typename... A>
static void launch_smem(void (*kernel)(P...), uint32_t blocks, int threads, int smem, cudaStream_t s, bool pdl, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename... P, typename... A>
static void launch(void (*kernel)(P...), uint32_t blocks, int threads, cudaStream_t s, bool pdl, A... args) {
  launch_smem(kernel, blocks, threads, 0, s, pdl, args...);
}

// Where a launch finds its descriptors: by value in the kernel parameters (`ld`), or in a table in global memory.
struct DescSource {
  const LaunchDesc *ld;  // non-null: parameter path
  const DevPiece *table;
};

#define AMAP_LAUNCH(KO, KP, KT, threads, ...)                                                          \
  do {                                                                                                 \
    if (ds.ld && ds.ld->n_pieces == 1) launch(KO<__VA_ARGS__>, L.n_blocks, threads, s, pdl, ds.ld->piece[0], pt); \
    else if (ds.ld) launch(KP<__VA_ARGS__>, L.n_blocks, threads, s, pdl, *ds.ld, pt);                  \
    else launch(KT<__VA_ARGS__>, L.n_blocks, threads, s, pdl, ds.table, L.first_piece, L.n_pieces, pt); \
  } while (0)

template <int V>
static void launch_affine(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl) {
  if (L.cons > 2) {
    if (L.wide) AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, kDevMaxCons, int64_t);
    else AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, kDevMaxCons, uint32_t);
  } else if (L.cons > 0) {
    if (L.wide) AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, 2, int64_t);
    else AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, 2, uint32_t);
  } else {
    if (L.wide) AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, 0, int64_t);
    else AMAP_LAUNCH(amap_affine_one, amap_affine_param, amap_affine_table, kAffineThreads, V, kUnroll, 0, uint32_t);
  }
}

template <int V>
static void launch_strip(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl) {
  if (L.cons > 2) {
    if (L.wide) AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, kDevMaxCons, int64_t);
    else AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, kDevMaxCons, uint32_t);
  } else if (L.cons > 0) {
    if (L.wide) AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, 2, int64_t);
    else AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, 2, uint32_t);
  } else {
    if (L.wide) AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, 0, int64_t);
    else AMAP_LAUNCH(amap_strip_one, amap_strip_param, amap_strip_table, kAffineThreads, V, 0, uint32_t);
  }
}

template <int ES, int UB>
static void launch_transpose_narrow(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl) {
  if constexpr (UB >= ES && UB < 16) {
    if (L.wide) AMAP_LAUNCH(amap_transpose_narrow_one, amap_transpose_narrow_param, amap_transpose_narrow_table, kTransposeThreads, ES, UB, int64_t);
    else AMAP_LAUNCH(amap_transpose_narrow_one, amap_transpose_narrow_param, amap_transpose_narrow_table, kTransposeThreads, ES, UB, uint32_t);
  }
}

// The flat kernels: dynamic shared memory above the default limit has to be allowed per function (an attribute of
// the function in the current device's context).  Done when a plan with such launches is made for a device and on
// the first amap_execute_static on a device, never while launches are enqueued.
template <int ES, int T>
static cudaError_t allow_flat_panels_for() {
  cudaError_t e = cudaSuccess;
  auto allow = [&](auto kernel) {
    const cudaError_t r = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFlatMaxPanelBytes);
    if (e == cudaSuccess) e = r;
  };
  allow(amap_transpose_flat_one<ES, T, false>);
  allow(amap_transpose_flat_param<ES, T, false>);
  allow(amap_transpose_flat_table<ES, T, false>);
  if constexpr (ES == 2) {
    allow(amap_transpose_flat_one<ES, T, true>);
    allow(amap_transpose_flat_param<ES, T, true>);
    allow(amap_transpose_flat_table<ES, T, true>);
  }
  allow(amap_transpose_flat_source_one<ES, T>);
  allow(amap_transpose_flat_source_param<ES, T>);
  allow(amap_transpose_flat_source_table<ES, T>);
  return e;
}
static cudaError_t allow_flat_panels() {
  cudaError_t e = allow_flat_panels_for<2, 256>();
  if (e == cudaSuccess) e = allow_flat_panels_for<2, 512>();
  if (e == cudaSuccess) e = allow_flat_panels_for<4, 256>();
  if (e == cudaSuccess) e = allow_flat_panels_for<4, 512>();
  return e;
}
static bool has_flat_launches(const amap_plan_t *plan) {
  for (const Launch &L : plan->launches)
    if (L.kind == kDevTranspose && L.cons <= -2) return true;
  return false;
}

template <int ES>
static void launch_transpose_flat(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl,
                                  bool source_side) {
  if constexpr (ES == 2 || ES == 4) {
    auto pick = [&](auto threads) {
      constexpr int T = decltype(threads)::value;
      if (source_side) {
        if (ds.ld && ds.ld->n_pieces == 1) launch_smem(amap_transpose_flat_source_one<ES, T>, L.n_blocks, T, L.smem, s, pdl, ds.ld->piece[0], pt);
        else if (ds.ld) launch_smem(amap_transpose_flat_source_param<ES, T>, L.n_blocks, T, L.smem, s, pdl, *ds.ld, pt);
        else launch_smem(amap_transpose_flat_source_table<ES, T>, L.n_blocks, T, L.smem, s, pdl, ds.table, L.first_piece, L.n_pieces, pt);
      } else if (ES == 2 && L.paired) {
        constexpr bool P = ES == 2;
        if (ds.ld && ds.ld->n_pieces == 1) launch_smem(amap_transpose_flat_one<ES, T, P>, L.n_blocks, T, L.smem, s, pdl, ds.ld->piece[0], pt);
        else if (ds.ld) launch_smem(amap_transpose_flat_param<ES, T, P>, L.n_blocks, T, L.smem, s, pdl, *ds.ld, pt);
        else launch_smem(amap_transpose_flat_table<ES, T, P>, L.n_blocks, T, L.smem, s, pdl, ds.table, L.first_piece, L.n_pieces, pt);
      } else {
        if (ds.ld && ds.ld->n_pieces == 1) launch_smem(amap_transpose_flat_one<ES, T, false>, L.n_blocks, T, L.smem, s, pdl, ds.ld->piece[0], pt);
        else if (ds.ld) launch_smem(amap_transpose_flat_param<ES, T, false>, L.n_blocks, T, L.smem, s, pdl, *ds.ld, pt);
        else launch_smem(amap_transpose_flat_table<ES, T, false>, L.n_blocks, T, L.smem, s, pdl, ds.table, L.first_piece, L.n_pieces, pt);
      }
    };
    if (L.threads == 512) pick(std::integral_constant<int, 512>());
    else pick(std::integral_constant<int, 256>());
  }
}

template <int ES>
static void launch_transpose(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl) {
  switch (L.cons) {  // access width of the launch
    case -2: launch_transpose_flat<ES>(ds, L, pt, s, pdl, false); return;
    case -3: launch_transpose_flat<ES>(ds, L, pt, s, pdl, true); return;
    case -1:
      if constexpr (ES <= 4)
        AMAP_LAUNCH(amap_transpose_realign_one, amap_transpose_realign_param, amap_transpose_realign_table, kTransposeThreads, ES);
      return;
    case 0:
      if constexpr (ES <= 4) AMAP_LAUNCH(amap_transpose_shifted_one, amap_transpose_shifted_param, amap_transpose_shifted_table, kTransposeThreads, ES);
      return;
    case 8: launch_transpose_narrow<ES, 8>(ds, L, pt, s, pdl); return;
    case 4: launch_transpose_narrow<ES, 4>(ds, L, pt, s, pdl); return;
    case 2: launch_transpose_narrow<ES, 2>(ds, L, pt, s, pdl); return;
    case 1: launch_transpose_narrow<ES, 1>(ds, L, pt, s, pdl); return;
    default: break;
  }
  if (L.wide) AMAP_LAUNCH(amap_transpose_one, amap_transpose_param, amap_transpose_table, kTransposeThreads, ES, int64_t);
  else AMAP_LAUNCH(amap_transpose_one, amap_transpose_param, amap_transpose_table, kTransposeThreads, ES, uint32_t);
}

static cudaError_t enqueue(const DescSource &ds, const Launch &L, const PtrTable &pt, cudaStream_t s, bool pdl) {
  if (L.kind == kDevStrip) {
    switch (L.unit) {
      case 16: launch_strip<16>(ds, L, pt, s, pdl); break;
      case 8: launch_strip<8>(ds, L, pt, s, pdl); break;
      case 4: launch_strip<4>(ds, L, pt, s, pdl); break;
      case 2: launch_strip<2>(ds, L, pt, s, pdl); break;
      default: launch_strip<1>(ds, L, pt, s, pdl); break;
    }
  } else if (L.kind == kDevTranspose) {
    switch (L.unit) {
      case 8: launch_transpose<8>(ds, L, pt, s, pdl); break;
      case 4: launch_transpose<4>(ds, L, pt, s, pdl); break;
      case 2: launch_transpose<2>(ds, L, pt, s, pdl); break;
      default: launch_transpose<1>(ds, L, pt, s, pdl); break;
    }
  } else {
    switch (L.unit) {
      case 16: launch_affine<16>(ds, L, pt, s, pdl); break;
      case 8: launch_affine<8>(ds, L, pt, s, pdl); break;
      case 4: launch_affine<4>(ds, L, pt, s, pdl); break;
      case 2: launch_affine<2>(ds, L, pt, s, pdl); break;
      default: launch_affine<1>(ds, L, pt, s, pdl); break;
    }
  }
  return cudaGetLastError();
}

// Argument checks shared by the execute entry points: null pointers, alignment to the plan's pointer_align, and no
// overlap between the byte ranges of any two buffers of which one is written.  Fills pt->src for the external
// inputs and pt->dst for the outputs.
static int bind_buffers(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *const *dst_dev_ptrs, PtrTable *pt) {
  if (!src_dev_ptrs && !plan->in_numel.empty()) return AMAP_EINVAL;
  if (!dst_dev_ptrs) return AMAP_EINVAL;
  memset(pt, 0, sizeof *pt);
  const uintptr_t mask = (uintptr_t)plan->pointer_align - 1;
  const size_t n_out = plan->out_numels.size();
  for (size_t k = 0; k < n_out; ++k) {
    if (!dst_dev_ptrs[k] && plan->out_numels[k] > 0) return AMAP_EINVAL;
    const uintptr_t d0 = (uintptr_t)dst_dev_ptrs[k], d1 = d0 + (uintptr_t)plan->out_numels[k] * plan->elem_size;
    if (d0 & mask) return AMAP_EALIGN;
    for (size_t j = 0; j < k; ++j) {  // two outputs must not overlap either
      const uintptr_t e0 = (uintptr_t)dst_dev_ptrs[j], e1 = e0 + (uintptr_t)plan->out_numels[j] * plan->elem_size;
      if (d0 < e1 && e0 < d1) return AMAP_EINVAL;
    }
    pt->set_dst((int)k, (char *)dst_dev_ptrs[k]);
  }
  for (size_t q = 0; q < plan->in_numel.size(); ++q) {
    if (!src_dev_ptrs[q]) {  // allowed for an input that no piece of this map reads
      if (plan->in_used[q] && plan->in_numel[q] > 0) return AMAP_EINVAL;
      continue;
    }
    if ((uintptr_t)src_dev_ptrs[q] & mask) return AMAP_EALIGN;
    const uintptr_t s0 = (uintptr_t)src_dev_ptrs[q], s1 = s0 + (uintptr_t)plan->in_numel[q] * plan->elem_size;
    for (size_t k = 0; k < n_out; ++k) {  // source and destination ranges must not overlap
      const uintptr_t d0 = (uintptr_t)dst_dev_ptrs[k], d1 = d0 + (uintptr_t)plan->out_numels[k] * plan->elem_size;
      if (s0 < d1 && d0 < s1) return AMAP_EINVAL;
    }
    pt->src[q] = (const char *)src_dev_ptrs[q];
  }
  return AMAP_OK;
}

static bool nothing_to_write(const amap_plan_t *plan) {
  for (int64_t n : plan->out_numels)
    if (n > 0) return false;
  return true;
}

extern "C" int amap_execute_multi(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *const *dst_dev_ptrs,
                                  void *cuda_stream) {
  if (!plan || plan->device < 0) return AMAP_EINVAL;
  if (nothing_to_write(plan)) return AMAP_OK;
  PtrTable pt;
  const int brc = bind_buffers(plan, src_dev_ptrs, dst_dev_ptrs, &pt);
  if (brc != AMAP_OK) return brc;
  const size_t n_in = plan->in_numel.size();
  for (size_t k = 0; k < plan->temps.size(); ++k) pt.src[n_in + k] = (const char *)plan->temps[k];
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int prev = 0;
  CUDA_TRY(cudaGetDevice(&prev));
  if (prev != plan->device) CUDA_TRY(cudaSetDevice(plan->device));
  struct Restore {
    int prev, cur;
    ~Restore() { if (prev != cur) cudaSetDevice(prev); }
  } restore{prev, plan->device};
  for (size_t li = 0; li < plan->launches.size(); ++li) {
    const Launch &L = plan->launches[li];
    const LaunchDesc &ld = plan->launch_desc[li];
    const int t = plan->stage_dst[L.stage];
    PtrTable stage_pt = pt;  // stages run in stream order; a stage that writes a temporary has one destination
    if (t >= 0) stage_pt.set_dst(0, (char *)plan->temps[t]);
    const DescSource ds{ld.n_pieces > 0 ? &ld : nullptr, plan->dev_table};
    const cudaError_t e = enqueue(ds, L, stage_pt, s, plan->pdl);
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute: kernel launch");
  }
  return AMAP_OK;
}

extern "C" int amap_execute(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr,
                            void *cuda_stream) {
  if (!plan || plan->out_numels.size() != 1) return AMAP_EINVAL;
  if (plan->out_numel == 0) return AMAP_OK;
  if (!dst_dev_ptr) return AMAP_EINVAL;
  void *dsts[1] = {dst_dev_ptr};
  return amap_execute_multi(plan, src_dev_ptrs, dsts, cuda_stream);
}

extern "C" int amap_execute_host(amap_plan_t *plan, const void *const *src_host_ptrs, void *dst_host_ptr,
                                 void *cuda_stream) {
  if (!plan || plan->device < 0 || plan->out_numels.size() != 1 || (!src_host_ptrs && !plan->in_numel.empty()) ||
      (!dst_host_ptr && plan->out_numel > 0))
    return AMAP_EINVAL;
  int prev = 0;
  CUDA_TRY(cudaGetDevice(&prev));
  CUDA_TRY(cudaSetDevice(plan->device));
  const size_t es = (size_t)plan->elem_size;
  int rc = AMAP_OK;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaSuccess;
  if (plan->stage_in.empty() && !plan->in_numel.empty()) plan->stage_in.assign(plan->in_numel.size(), nullptr);
  for (size_t q = 0; q < plan->in_numel.size() && e == cudaSuccess; ++q)
    if (!plan->stage_in[q] && plan->in_numel[q] > 0) e = cudaMalloc(&plan->stage_in[q], plan->in_numel[q] * es);
  if (e == cudaSuccess && !plan->stage_out && plan->out_numel > 0) e = cudaMalloc(&plan->stage_out, plan->out_numel * es);
  if (e == cudaSuccess && plan->slab_plan && plan->events.empty()) {  // the pipeline's streams and events, once
    e = cudaStreamCreateWithFlags(&plan->h2d_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&plan->d2h_stream, cudaStreamNonBlocking);
    for (int k = 0; k < 2 * plan->n_slabs + 2 && e == cudaSuccess; ++k) {
      cudaEvent_t ev;
      e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
      if (e == cudaSuccess) plan->events.push_back(ev);
    }
  }
  if (e == cudaSuccess && plan->slab_plan) {
    // upload slab k+1 while slab k runs and slab k-1 downloads; the caller's stream carries the kernels
    const int S = plan->n_slabs;
    cudaEvent_t *ev = plan->events.data();
    e = cudaEventRecord(ev[0], s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(plan->h2d_stream, ev[0], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(plan->d2h_stream, ev[0], 0);
    std::vector<const void *> srcs(plan->in_numel.size());
    for (int k = 0; k < S && e == cudaSuccess && rc == AMAP_OK; ++k) {
      for (size_t q = 0; q < plan->in_numel.size() && e == cudaSuccess; ++q) {
        const size_t off = (size_t)k * plan->slab_in_bytes[q];
        srcs[q] = (const char *)plan->stage_in[q] + off;
        if (plan->slab_in_bytes[q] > 0)
          e = cudaMemcpyAsync((char *)plan->stage_in[q] + off, (const char *)src_host_ptrs[q] + off, plan->slab_in_bytes[q],
                              cudaMemcpyHostToDevice, plan->h2d_stream);
      }
      if (e == cudaSuccess) e = cudaEventRecord(ev[1 + 2 * k], plan->h2d_stream);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ev[1 + 2 * k], 0);
      char *out_k = (char *)plan->stage_out + (size_t)k * plan->slab_out_bytes;
      if (e == cudaSuccess) rc = amap_execute(plan->slab_plan, srcs.data(), out_k, cuda_stream);
      if (e == cudaSuccess && rc == AMAP_OK) e = cudaEventRecord(ev[2 + 2 * k], s);
      if (e == cudaSuccess && rc == AMAP_OK) e = cudaStreamWaitEvent(plan->d2h_stream, ev[2 + 2 * k], 0);
      if (e == cudaSuccess && rc == AMAP_OK)
        e = cudaMemcpyAsync((char *)dst_host_ptr + (size_t)k * plan->slab_out_bytes, out_k, plan->slab_out_bytes,
                            cudaMemcpyDeviceToHost, plan->d2h_stream);
    }
    if (e == cudaSuccess) e = cudaEventRecord(ev[2 * S + 1], plan->d2h_stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ev[2 * S + 1], 0);
    // always drain what was enqueued, also after an error, before the buffers can be reused
    cudaStreamSynchronize(plan->h2d_stream);
    cudaStreamSynchronize(plan->d2h_stream);
    const cudaError_t e2 = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = e2;
    cudaSetDevice(prev);
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute_host");
    return rc;
  }
  for (size_t q = 0; q < plan->in_numel.size() && e == cudaSuccess; ++q)
    if (plan->in_numel[q] > 0)
      e = cudaMemcpyAsync(plan->stage_in[q], src_host_ptrs[q], plan->in_numel[q] * es, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) {
    rc = amap_execute(plan, (const void *const *)plan->stage_in.data(), plan->stage_out, cuda_stream);
    if (rc == AMAP_OK && plan->out_numel > 0)
      e = cudaMemcpyAsync(dst_host_ptr, plan->stage_out, plan->out_numel * es, cudaMemcpyDeviceToHost, s);
    if (rc == AMAP_OK && e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  cudaSetDevice(prev);
  if (e != cudaSuccess) return cuda_fail(e, "amap_execute_host");
  return rc;
}

// ---------------------------------------------------------------------------
// amap_execute_static: the same copy for callers that must not allocate.
// The descriptor table, which amap_plan normally places in memory it gets from
// cudaMalloc, is kept in a fixed array inside the library image instead.
// ---------------------------------------------------------------------------
static const int kStaticMaxPieces = 64;
static __device__ __align__(256) unsigned char g_static_table[kStaticMaxPieces * sizeof(DevPiece)];

// writes descriptors [first, first + ld.n_pieces) of the fixed array (device code names the array directly)
__global__ void amap_static_table_store(const __grid_constant__ LaunchDesc ld, int first) {
  const uint32_t *src = reinterpret_cast<const uint32_t *>(ld.piece);
  uint32_t *dst = reinterpret_cast<uint32_t *>(g_static_table + (size_t)first * sizeof(DevPiece));
  const int words = ld.n_pieces * (int)(sizeof(DevPiece) / 4);
  for (int w = threadIdx.x; w < words; w += blockDim.x) dst[w] = src[w];
}

static const int kStaticMaxDevices = 64;
static void *g_static_table_addr[kStaticMaxDevices];  // device address of g_static_table, per device, 0 = not set up

// In host code `g_static_table` is only a handle for the runtime; the address the
// kernels need comes from cudaGetSymbolAddress, once per device, with that device current.
static int static_table_address(int device, void **out) {
  if (device < 0 || device >= kStaticMaxDevices) return AMAP_EINVAL;
  void *p = __atomic_load_n(&g_static_table_addr[device], __ATOMIC_ACQUIRE);
  if (!p) {
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_table);
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute_static: cudaGetSymbolAddress");
    if (!p) return AMAP_ECUDA;
    __atomic_store_n(&g_static_table_addr[device], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return AMAP_OK;
}

// multiprocessors of the current device, looked up once per device (the look-ahead distance of a dry plan is
// set for the device the call runs on)
static char g_static_flat_allowed[kStaticMaxDevices];  // the flat kernels' shared-memory attribute is set on the device
static int g_static_sms[kStaticMaxDevices];
static int static_device_sms(int device) {
  int n = __atomic_load_n(&g_static_sms[device], __ATOMIC_ACQUIRE);
  if (n <= 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = kDefaultSms;
    __atomic_store_n(&g_static_sms[device], n, __ATOMIC_RELEASE);
  }
  return n;
}

extern "C" int amap_execute_static(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr,
                                   void *cuda_stream) {
  if (!plan || plan->out_numels.size() != 1) return AMAP_EINVAL;
  if (plan->table.size() > (size_t)kStaticMaxPieces) return AMAP_ETOOLARGE;
  if (!plan->temp_numel.empty()) return AMAP_EUNSUPPORTED;  // temporaries would need device memory
  if (plan->out_numel == 0) return AMAP_OK;
  PtrTable pt;
  void *dsts[1] = {dst_dev_ptr};
  const int brc = bind_buffers(plan, src_dev_ptrs, dsts, &pt);  // the same refusals as amap_execute
  if (brc != AMAP_OK) return brc;
  int device = 0;
  CUDA_TRY(cudaGetDevice(&device));
  if (plan->device >= 0 && plan->device != device) return AMAP_EINVAL;
  void *table = nullptr;
  const int rc = static_table_address(device, &table);
  if (rc != AMAP_OK) return rc;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  // The descriptors travel to the array in the parameters of small kernels, kParamPieces at a time: nothing is
  // copied from host memory, so neither the host nor the stream is made to wait.  A dry plan was made without
  // knowing the device: its look-ahead distances assume kDefaultSms multiprocessors and are rescaled here.
  const int sms = static_device_sms(device);
  const bool rescale = plan->device < 0 && sms != kDefaultSms;
  if (has_flat_launches(plan) && device < kStaticMaxDevices && !g_static_flat_allowed[device]) {
    CUDA_TRY(allow_flat_panels());
    g_static_flat_allowed[device] = 1;
  }
  for (size_t first = 0; first < plan->table.size(); first += kParamPieces) {
    LaunchDesc ld;
    memset(&ld, 0, sizeof ld);
    ld.n_pieces = (int32_t)std::min<size_t>(kParamPieces, plan->table.size() - first);
    for (int q = 0; q < ld.n_pieces; ++q) {
      ld.piece[q] = plan->table[first + q];
      if (rescale && ld.piece[q].prefetch > 1)
        ld.piece[q].prefetch = std::max(2, (int)((int64_t)ld.piece[q].prefetch * sms / kDefaultSms));
    }
    // a plain launch: it starts only after everything before it on the stream (an earlier call's kernels, which
    // still read the array) has finished
    amap_static_table_store<<<1, 256, 0, s>>>(ld, (int)first);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute_static: descriptor upload");
  }
  bool first_launch = true;
  for (const Launch &L : plan->launches) {
    const DescSource ds{nullptr, (const DevPiece *)table};  // always through the fixed table
    // The first copy kernel must not start before the upload kernels have completed (it reads its descriptor ahead
    // of its grid-dependency wait), so it is launched without programmatic dependent launch; the later ones only
    // follow kernels that leave the array alone.
    const cudaError_t e = enqueue(ds, L, pt, s, plan->pdl && !first_launch);
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute_static: kernel launch");
    first_launch = false;
  }
  return AMAP_OK;
}
