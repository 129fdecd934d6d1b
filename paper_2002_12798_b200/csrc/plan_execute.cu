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
  int kind;       // DevKind
  int unit;       // bytes per item (affine kernel) / element size (transpose)
  int first_piece;
  int n_pieces;
  uint32_t n_blocks;
};

struct amap_plan_t {
  int device = 0;
  int elem_size = 0;
  int pointer_align = 0;
  std::vector<int64_t> in_numel;
  int64_t out_numel = 0;
  std::vector<DevPiece> table;
  std::vector<int> piece_kernel;  // amap_kernel_kind per map piece
  std::vector<Launch> launches;
  DevPiece *dev_table = nullptr;
  amap_stats stats;
  // staging for amap_execute_host (allocated on first use)
  std::vector<void *> stage_in;
  void *stage_out = nullptr;
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

static const int kUnroll = 8;  // units per thread in the affine kernel

// largest power-of-two unit (<= 16 bytes) in which the piece is still an affine loop nest
static int pick_unit(const Piece &p, int es, int ptr_align, int force_kind) {
  if (force_kind == AMAP_KERNEL_GATHER) return es;
  const int n = p.n();
  if (n == 0) return es;
  const int in = n - 1;  // canonical order: innermost destination loop last
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
  d->n_guards = (int)p.guards.size();
  d->n_domain = (int)p.domain.size();
  int c = 0;
  auto put = [&](const Con &g) -> bool {
    d->cons[c].off = g.e.c0;
    d->cons[c].extent = g.extent;
    for (size_t j = 0; j < loops.size(); ++j) {
      const int64_t v = g.e.c[loops[j]];
      if (v > INT32_MAX || v < INT32_MIN) return false;
      d->cons[c].coef[j] = (int32_t)v;
    }
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
  bool load = d.input >= 0, live = true;
  for (int c = 0; c < nc; ++c) {
    const int64_t v = acc[c] + d.cons[c].off;
    const bool ok = v >= 0 && v < d.cons[c].extent;
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

extern "C" int amap_plan(const amap_map *map, int device, const amap_plan_opts *opts, amap_plan_t **out_plan) {
  if (!map || !out_plan) return AMAP_EINVAL;
  amap_plan_opts o;
  memset(&o, 0, sizeof o);
  if (opts) o = *opts;
  for (int r : o.reserved)
    if (r != 0) return AMAP_EINVAL;
  if (o.force_kernel < AMAP_KERNEL_AUTO || o.force_kernel > AMAP_KERNEL_FILL) return AMAP_EINVAL;
  const Map &m = map->m;
  const int es = m.elem_size;
  int align = o.pointer_align ? o.pointer_align : es;
  if (align < es || (align & (align - 1))) return AMAP_EINVAL;
  if ((int)m.in_numel.size() > kMaxInputs) return AMAP_EUNSUPPORTED;

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
  pl->in_numel = m.in_numel;
  pl->out_numel = m.out_numel;
  memset(&pl->stats, 0, sizeof pl->stats);
  pl->stats.n_pieces = (int32_t)m.pieces.size();

  // one launch of the affine kernel per unit width present (pieces grouped by width)
  std::vector<int> unit_of(m.pieces.size());
  std::vector<int64_t> reads(m.in_numel.size(), 0);
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
      reads[p.src] += piece_unique_reads(p, m.in_numel[p.src]);
      kind = (unit_of[q] > es || (p.n() > 0 && p.srcoff.c[p.n() - 1] == 1 && p.dst.c[p.n() - 1] == 1)) ? AMAP_KERNEL_COPY
                                                                                                         : AMAP_KERNEL_GATHER;
    }
    pl->piece_kernel.push_back(kind);
  }
  for (size_t q = 0; q < reads.size(); ++q) pl->stats.bytes_read += std::min(reads[q], m.in_numel[q]) * es;

  for (int V = 16; V >= 1; V >>= 1) {
    Launch L{kDevAffine, V, (int)pl->table.size(), 0, 0};
    for (size_t q = 0; q < m.pieces.size(); ++q) {
      if (unit_of[q] != V) continue;
      DevPiece d;
      const int rc = build_affine_piece(m.pieces[q], es, V, &d);
      if (rc != AMAP_OK) {
        delete pl;
        return rc;
      }
      if (d.n_items == 0) continue;
      const int64_t in_bytes = (d.input >= 0) ? m.in_numel[d.input] * es : 0;
      if (!check_affine_piece(d, in_bytes, m.out_numel * es)) {
        if (getenv("AMAP_LOG")) fprintf(stderr, "[amap] plan self-check failed on piece %zu\n", q);
        delete pl;
        return AMAP_EOVERFLOW;
      }
      if ((uint64_t)L.n_blocks + d.n_blocks > 0x7FFFFFFFull) {
        delete pl;
        return AMAP_EUNSUPPORTED;
      }
      d.first_block = L.n_blocks;
      L.n_blocks += d.n_blocks;
      L.n_pieces++;
      pl->table.push_back(d);
    }
    if (L.n_pieces > 0) pl->launches.push_back(L);
  }
  for (int k : pl->piece_kernel) {
    const int slot = (k == AMAP_KERNEL_GATHER) ? 0 : (k == AMAP_KERNEL_COPY) ? 1 : (k == AMAP_KERNEL_TRANSPOSE) ? 2 : 3;
    pl->stats.kernel_kind[slot]++;
  }
  pl->stats.n_launches = (int32_t)pl->launches.size();

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
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    if (pl->dev_table) cudaFree(pl->dev_table);
    delete pl;
    return cuda_fail(e, "amap_plan: descriptor table upload");
  }
  *out_plan = pl;
  return AMAP_OK;
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
  for (void *p : plan->stage_in)
    if (p) cudaFree(p);
  if (plan->stage_out) cudaFree(plan->stage_out);
  cudaSetDevice(prev);
  delete plan;
}

extern "C" int amap_plan_stats(const amap_plan_t *plan, amap_stats *out) {
  if (!plan || !out) return AMAP_EINVAL;
  *out = plan->stats;
  return AMAP_OK;
}

extern "C" int amap_plan_piece_kernel(const amap_plan_t *plan, int32_t k, int32_t *kind) {
  if (!plan || !kind || k < 0 || k >= (int32_t)plan->piece_kernel.size()) return AMAP_EINVAL;
  *kind = plan->piece_kernel[k];
  return AMAP_OK;
}

template <int V>
static cudaError_t launch_affine(const amap_plan_t *pl, const Launch &L, const PtrTable &pt, cudaStream_t s) {
  amap_affine_kernel<V, kUnroll><<<L.n_blocks, kAffineThreads, 0, s>>>(pl->dev_table, L.first_piece, L.n_pieces, pt);
  return cudaGetLastError();
}

extern "C" int amap_execute(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr,
                            void *cuda_stream) {
  if (!plan || plan->device < 0 || (!src_dev_ptrs && !plan->in_numel.empty())) return AMAP_EINVAL;
  if (plan->out_numel == 0) return AMAP_OK;
  if (!dst_dev_ptr) return AMAP_EINVAL;
  PtrTable pt;
  memset(&pt, 0, sizeof pt);
  const uintptr_t mask = (uintptr_t)plan->pointer_align - 1;
  for (size_t q = 0; q < plan->in_numel.size(); ++q) {
    if (!src_dev_ptrs[q] && plan->in_numel[q] > 0) return AMAP_EINVAL;
    if ((uintptr_t)src_dev_ptrs[q] & mask) return AMAP_EALIGN;
    if (src_dev_ptrs[q] == dst_dev_ptr) return AMAP_EINVAL;
    pt.src[q] = (const char *)src_dev_ptrs[q];
  }
  if ((uintptr_t)dst_dev_ptr & mask) return AMAP_EALIGN;
  pt.dst = (char *)dst_dev_ptr;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int prev = 0;
  CUDA_TRY(cudaGetDevice(&prev));
  if (prev != plan->device) CUDA_TRY(cudaSetDevice(plan->device));
  struct Restore {
    int prev, cur;
    ~Restore() { if (prev != cur) cudaSetDevice(prev); }
  } restore{prev, plan->device};
  for (const Launch &L : plan->launches) {
    cudaError_t e = cudaSuccess;
    switch (L.unit) {
      case 16: e = launch_affine<16>(plan, L, pt, s); break;
      case 8: e = launch_affine<8>(plan, L, pt, s); break;
      case 4: e = launch_affine<4>(plan, L, pt, s); break;
      case 2: e = launch_affine<2>(plan, L, pt, s); break;
      default: e = launch_affine<1>(plan, L, pt, s); break;
    }
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute: kernel launch");
  }
  return AMAP_OK;
}

extern "C" int amap_execute_host(amap_plan_t *plan, const void *const *src_host_ptrs, void *dst_host_ptr,
                                 void *cuda_stream) {
  if (!plan || plan->device < 0 || (!src_host_ptrs && !plan->in_numel.empty()) || (!dst_host_ptr && plan->out_numel > 0))
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

template <int V>
static cudaError_t launch_affine_at(const DevPiece *table, const Launch &L, const PtrTable &pt, cudaStream_t s) {
  amap_affine_kernel<V, kUnroll><<<L.n_blocks, kAffineThreads, 0, s>>>(table, L.first_piece, L.n_pieces, pt);
  return cudaGetLastError();
}

extern "C" int amap_execute_static(const amap_plan_t *plan, const void *const *src_dev_ptrs, void *dst_dev_ptr,
                                   void *cuda_stream) {
  if (!plan || (!src_dev_ptrs && !plan->in_numel.empty())) return AMAP_EINVAL;
  if (plan->table.size() > (size_t)kStaticMaxPieces) return AMAP_ETOOLARGE;
  if (plan->out_numel == 0) return AMAP_OK;
  if (!dst_dev_ptr) return AMAP_EINVAL;
  PtrTable pt;
  memset(&pt, 0, sizeof pt);
  const uintptr_t mask = (uintptr_t)plan->pointer_align - 1;
  for (size_t q = 0; q < plan->in_numel.size(); ++q) {
    if (!src_dev_ptrs[q] && plan->in_numel[q] > 0) return AMAP_EINVAL;
    if ((uintptr_t)src_dev_ptrs[q] & mask) return AMAP_EALIGN;
    if (src_dev_ptrs[q] == dst_dev_ptr) return AMAP_EINVAL;
    pt.src[q] = (const char *)src_dev_ptrs[q];
  }
  if ((uintptr_t)dst_dev_ptr & mask) return AMAP_EALIGN;
  pt.dst = (char *)dst_dev_ptr;
  int device = 0;
  CUDA_TRY(cudaGetDevice(&device));
  if (plan->device >= 0 && plan->device != device) return AMAP_EINVAL;
  void *table = nullptr;
  const int rc = static_table_address(device, &table);
  if (rc != AMAP_OK) return rc;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  // the part of the array this plan uses is overwritten in full; nothing in it needs to start at zero
  CUDA_TRY(cudaMemcpyAsync(table, plan->table.data(), plan->table.size() * sizeof(DevPiece), cudaMemcpyHostToDevice, s));
  for (const Launch &L : plan->launches) {
    cudaError_t e = cudaSuccess;
    const DevPiece *t = (const DevPiece *)table;
    switch (L.unit) {
      case 16: e = launch_affine_at<16>(t, L, pt, s); break;
      case 8: e = launch_affine_at<8>(t, L, pt, s); break;
      case 4: e = launch_affine_at<4>(t, L, pt, s); break;
      case 2: e = launch_affine_at<2>(t, L, pt, s); break;
      default: e = launch_affine_at<1>(t, L, pt, s); break;
    }
    if (e != cudaSuccess) return cuda_fail(e, "amap_execute_static: kernel launch");
  }
  return AMAP_OK;
}
