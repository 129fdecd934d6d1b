// Device code of the surviving copy (the data movement that Section 2.1 of the
// paper cannot remove and Section 2.2 wants run at full memory bandwidth).
// Pure data movement: no tensor cores, no floating-point arithmetic.
#pragma once
#include <cuda_runtime.h>

#include "device_table.hpp"

namespace amap {

template <int V> struct Unit;
template <> struct Unit<1> { using T = uint8_t; };
template <> struct Unit<2> { using T = uint16_t; };
template <> struct Unit<4> { using T = uint32_t; };
template <> struct Unit<8> { using T = uint2; };
template <> struct Unit<16> { using T = uint4; };

// Programmatic dependent launch: let the next kernel on the stream start its
// prologue now; wait (before touching any caller buffer) until the kernel
// before this one has completed and its writes are visible.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Compiler-only fence: read-only (non-coherent) loads may otherwise be sunk below later stores, which would
// serialise the requests a thread is meant to keep in flight together.
__device__ __forceinline__ void issue_barrier() { asm volatile("" ::: "memory"); }

__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv &f) {
  const uint32_t t = __umulhi(f.mul, n);
  return (t + ((n - t) >> f.sh1)) >> f.sh2;
}

template <int V>
__device__ __forceinline__ typename Unit<V>::T fill_unit(const DevPiece &p) {
  typename Unit<V>::T v;
  if constexpr (V == 16) {
    v = make_uint4((uint32_t)p.fill[0], (uint32_t)(p.fill[0] >> 32), (uint32_t)p.fill[1], (uint32_t)(p.fill[1] >> 32));
  } else if constexpr (V == 8) {
    v = make_uint2((uint32_t)p.fill[0], (uint32_t)(p.fill[0] >> 32));
  } else {
    v = (typename Unit<V>::T)p.fill[0];
  }
  return v;
}

// Read-only global load.  Written as volatile PTX so that the compiler keeps the loads of a thread together,
// ahead of the issue_barrier() that follows them (an intrinsic load could be sunk below later stores).
__device__ __forceinline__ uint4 load_16(const char *p) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <int V>
__device__ __forceinline__ typename Unit<V>::T load_unit(const char *p) {
  if constexpr (V == 16) {
    return load_16(p);
  } else if constexpr (V == 8) {
    uint2 v;
    asm volatile("ld.global.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
  } else if constexpr (V == 4) {
    uint32_t v;
    asm volatile("ld.global.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
  } else if constexpr (V == 2) {
    uint16_t v;
    asm volatile("ld.global.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
  } else {
    uint32_t v;
    asm volatile("ld.global.u8 %0, [%1];" : "=r"(v) : "l"(p));
    return (uint8_t)v;
  }
}

template <int V>
__device__ __forceinline__ void store_unit(char *p, typename Unit<V>::T v) {
  __stcs(reinterpret_cast<typename Unit<V>::T *>(p), v);
}

// find the piece a block belongs to and copy its descriptor to shared memory
__device__ __forceinline__ void fetch_piece(const DevPiece *__restrict__ table, int first_piece, int n_pieces,
                                            DevPiece *sp) {
  // the last piece whose first block is at or below this block's index: a binary search, since every probe is a
  // dependent load from global memory (a linear walk over 64 descriptors cost tens of microseconds per block)
  int p = first_piece, hi = first_piece + n_pieces - 1;
  while (p < hi) {
    const int mid = (p + hi + 1) >> 1;
    if (blockIdx.x >= table[mid].first_block) p = mid;
    else hi = mid - 1;
  }
  const uint32_t *src = reinterpret_cast<const uint32_t *>(table + p);
  uint32_t *dst = reinterpret_cast<uint32_t *>(sp);
  for (int w = threadIdx.x; w < (int)(sizeof(DevPiece) / 4); w += blockDim.x) dst[w] = src[w];
  __syncthreads();
}

// ---------------------------------------------------------------------------
// Affine copy: every thread moves U units of V bytes.  Unit L of a piece is
// decomposed into loop indices (innermost fastest), which give the source and
// destination byte offsets  b + sum_k stride_k * i_k  of the composed map.
// With V = 16 and a contiguous innermost loop this is the coalesced streaming
// copy; with V = elem_size and arbitrary strides it is the gather that handles
// every piece, including non-injective loads (overlapping windows) and guards
// (out-of-range loads give the fill value).  All U loads are issued before the
// first store so that each thread keeps U independent requests in flight; the
// loop over the nest is outermost so that each descriptor field is fetched
// once for the U units.
//   NC   : 0 = the piece has no constraints; otherwise the table's guards and
//          domain constraints (at most kDevMaxCons) are evaluated per unit.
//   OffT : uint32_t when every byte offset is below 4 GiB (wrap-around
//          arithmetic keeps intermediate negative values exact), else int64_t.
// ---------------------------------------------------------------------------
constexpr int kAffineThreads = 256;

template <int V, int U, int NC, typename OffT>
__device__ __forceinline__ void affine_body(const DevPiece &sp, const PtrTable &ptrs) {
  using T = typename Unit<V>::T;
  const int n = sp.n_loops;
  const uint64_t item0 = (uint64_t)(blockIdx.x - sp.first_block) * (uint64_t)(kAffineThreads * U) + threadIdx.x;
  const char *src = (sp.input >= 0) ? ptrs.src[sp.input] : nullptr;
  char *dst = ptrs.dst(sp.out);

  uint32_t rem[U], fu[U];
  OffT so[U], doff[U];
  bool live[U];
  int32_t acc[U][NC > 0 ? NC : 1];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const uint64_t L = item0 + (uint64_t)u * kAffineThreads;
    live[u] = L < sp.n_items;
    rem[u] = live[u] ? (uint32_t)L : 0u;
    fu[u] = sp.qa_f0;
    so[u] = (OffT)sp.soff;
    doff[u] = (OffT)sp.doff;
    if constexpr (NC > 0) {
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[u][c] = sp.cons[c].off;
    }
  }
  for (int k = n - 1; k >= 0; --k) {
    const FastDiv fd = sp.fd[k];
    const uint32_t ext = sp.ext[k];
    const OffT ss = (OffT)sp.sstride[k], ds = (OffT)sp.dstride[k];
    const uint32_t fs = sp.qa_fstride[k];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t q = fast_div(rem[u], fd);
      const uint32_t i = rem[u] - q * ext;
      rem[u] = q;
      so[u] += (OffT)i * ss;
      doff[u] += (OffT)i * ds;
      fu[u] += i * fs;  // the inner form of a quasi-affine source (all zero otherwise)
      if constexpr (NC > 0) {
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[u][c] += sp.cons[c].coef[k] * (int32_t)i;
      }
    }
  }
  if (sp.qa_n > 0) {  // block-uniform: split f into the digits of the statement that wrote the eliminated tensor
    for (int d = sp.qa_n - 1; d >= 0; --d) {
      const FastDiv fd = sp.qa_fd[d];
      const uint32_t radix = sp.qa_radix[d];
      const OffT st = (OffT)sp.qa_stride[d];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint32_t q = fast_div(fu[u], fd);
        so[u] += (OffT)(fu[u] - q * radix) * st;
        fu[u] = q;
      }
    }
  }
  bool load[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    load[u] = live[u] && (src != nullptr);
    if constexpr (NC > 0) {
      const int ng = sp.n_guards, nc = sp.n_guards + sp.n_domain;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const bool ok = (c >= nc) || ((uint32_t)acc[u][c] < (uint32_t)sp.cons[c].extent);
        if (c < ng) load[u] = load[u] && ok;  // a failed guard stores the fill value
        else live[u] = live[u] && ok;         // outside the piece's domain: nothing to do
      }
      load[u] = load[u] && live[u];
    }
  }
  T val[U];
  const T fill = fill_unit<V>(sp);
  // A contiguous piece (one loop of 16-byte units, a plain copy): the block's source bytes are one range.  While the
  // kernel before this one on the stream drains, ask L2 for them, and after the loads for the range of the block
  // that will take this block's place (`prefetch` blocks further on), as the transpose kernel does for its tiles.
  constexpr uint32_t kBlockBytes = kAffineThreads * U * V;
  const bool hint = V == 16 && NC == 0 && sp.prefetch && n == 1 && src != nullptr && sp.sstride[0] == V && threadIdx.x < 8;
  auto prefetch_block = [&](uint64_t block) {
    const uint64_t first = block * kBlockBytes + threadIdx.x * (kBlockBytes / 8), end = sp.n_items * V;
    if (first < end) {
      const uint32_t bytes = (uint32_t)min((uint64_t)(kBlockBytes / 8), end - first);
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + sp.soff + first), "r"(bytes) : "memory");
    }
  };
  if (hint) prefetch_block(blockIdx.x - sp.first_block);
  pdl_wait();
#pragma unroll
  for (int u = 0; u < U; ++u) val[u] = load[u] ? load_unit<V>(src + so[u]) : fill;
  issue_barrier();  // every load is issued before the first store
  if (hint && sp.prefetch > 1) prefetch_block((uint64_t)(blockIdx.x - sp.first_block) + (uint32_t)sp.prefetch);
#pragma unroll
  for (int u = 0; u < U; ++u)
    if (live[u]) store_unit<V>(dst + doff[u], val[u]);
}

// ---------------------------------------------------------------------------
// Strip copy: the affine copy for nests of two or more loops.  A thread
// decomposes ONE item index and then walks kStrip consecutive iterations of
// loop ku by adding that loop's strides, so the index arithmetic is paid once
// per kStrip units (a 3x3 window gather has six loops and two guards: per-unit
// decomposition would make it issue-bound).  Consecutive threads still take
// consecutive units of the innermost loop, so accesses stay coalesced, and all
// loads of a strip are issued before its first store.
// ---------------------------------------------------------------------------
template <int V, int NC, typename OffT>
__device__ __forceinline__ void strip_body(const DevPiece &sp, const PtrTable &ptrs) {
  using T = typename Unit<V>::T;
  const uint64_t item = (uint64_t)(blockIdx.x - sp.first_block) * kAffineThreads + threadIdx.x;
  if (item >= sp.n_items) return;
  const char *src = (sp.input >= 0) ? ptrs.src[sp.input] : nullptr;
  char *dst = ptrs.dst(sp.out);
  uint32_t rem = (uint32_t)item;
  OffT so = (OffT)sp.soff, dof = (OffT)sp.doff;
  int32_t acc[NC > 0 ? NC : 1];
  if constexpr (NC > 0) {
#pragma unroll
    for (int c = 0; c < NC; ++c) acc[c] = sp.cons[c].off;
  }
  uint32_t strip = 0;
  const int ku = sp.ku;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    const uint32_t q = fast_div(rem, sp.fd[k]);
    const uint32_t i = rem - q * sp.ext[k];
    rem = q;
    so += (OffT)i * (OffT)sp.sstride[k];
    dof += (OffT)i * (OffT)sp.dstride[k];
    if (k == ku) strip = i;
    if constexpr (NC > 0) {
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[c] += sp.cons[c].coef[k] * (int32_t)i;
    }
  }
  const uint32_t left = sp.ku_ext - strip * kStrip;  // iterations of loop ku that remain, >= 1
  const OffT ss = (OffT)sp.ku_ss, ds = (OffT)sp.ku_ds;
  bool live[kStrip], load[kStrip];
#pragma unroll
  for (int u = 0; u < kStrip; ++u) {
    live[u] = (uint32_t)u < left;
    load[u] = live[u] && (src != nullptr);
    if constexpr (NC > 0) {
      const int ng = sp.n_guards, nc = sp.n_guards + sp.n_domain;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const bool ok = (c >= nc) || ((uint32_t)(acc[c] + u * sp.ku_coef[c]) < (uint32_t)sp.cons[c].extent);
        if (c < ng) load[u] = load[u] && ok;
        else live[u] = live[u] && ok;
      }
      load[u] = load[u] && live[u];
    }
  }
  T val[kStrip];
  const T fill = fill_unit<V>(sp);
  pdl_wait();
#pragma unroll
  for (int u = 0; u < kStrip; ++u) val[u] = load[u] ? load_unit<V>(src + (OffT)(so + (OffT)u * ss)) : fill;
  issue_barrier();  // every load is issued before the first store
#pragma unroll
  for (int u = 0; u < kStrip; ++u)
    if (live[u]) store_unit<V>(dst + (OffT)(dof + (OffT)u * ds), val[u]);
}

// ---------------------------------------------------------------------------
// Tiled transpose for pieces whose destination-contiguous index a is not the
// source-contiguous index b.  A block moves a tile of (128 bytes of a) x
// (kTileB elements of b) = 16 KiB through shared memory:
//   phase 1  16-byte loads along b (full 128-byte lines of the source), stored
//            as 16-byte chunks in the row of their a;
//   phase 2  each thread gathers the 16/ES elements of 16/ES consecutive a at
//            one b, packs them, and stores 16 bytes along a (full lines of the
//            destination).
// The 16-byte chunk index within a row is XOR-ed with (a / (16/ES)) & 7, which
// spreads both the vector stores of phase 1 and the element reads of phase 2
// over all banks (a profiler capture of a full-size transpose still counts
// 1-2 % conflicting wavefronts, from the rounds of partly filled tiles).  Tiles
// on the ragged edge are predicated per chunk (the planner only selects this
// kernel when both extents are multiples of 16/ES).
// ---------------------------------------------------------------------------
// the 16-byte chunk index within a tile row is XOR-ed with this function of the row's chunk of a
template <int CA>
__device__ __forceinline__ int tile_swizzle(int ca) {
  return CA >= 8 ? (ca & 7) : ca * (8 / CA);
}

template <int ES, int CA = 8>
__device__ __forceinline__ uint4 gather_column(const unsigned char *tile, int ca, int b_l) {
  constexpr int EPU = 16 / ES;
  constexpr int RB = kTileB * ES * 8 / CA;
  const int chunk = b_l / EPU;
  const unsigned char *p = tile + (ca * EPU) * RB + ((chunk ^ tile_swizzle<CA>(ca)) << 4) + (b_l % EPU) * ES;
  uint4 out;
  if constexpr (ES == 1) {
    uint32_t w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      w[g] = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) w[g] |= (uint32_t)p[(g * 4 + j) * RB] << (8 * j);
    }
    out = make_uint4(w[0], w[1], w[2], w[3]);
  } else if constexpr (ES == 2) {
    uint32_t w[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const uint32_t lo = *reinterpret_cast<const uint16_t *>(p + (2 * g) * RB);
      const uint32_t hi = *reinterpret_cast<const uint16_t *>(p + (2 * g + 1) * RB);
      w[g] = lo | (hi << 16);
    }
    out = make_uint4(w[0], w[1], w[2], w[3]);
  } else if constexpr (ES == 4) {
    out.x = *reinterpret_cast<const uint32_t *>(p);
    out.y = *reinterpret_cast<const uint32_t *>(p + RB);
    out.z = *reinterpret_cast<const uint32_t *>(p + 2 * RB);
    out.w = *reinterpret_cast<const uint32_t *>(p + 3 * RB);
  } else {
    const uint2 lo = *reinterpret_cast<const uint2 *>(p);
    const uint2 hi = *reinterpret_cast<const uint2 *>(p + RB);
    out = make_uint4(lo.x, lo.y, hi.x, hi.y);
  }
  return out;
}

// A block of a fill piece (a strip or affine descriptor with 16-byte units, no source
// and no constraints) that rides in a transpose launch, so that a map made of
// transposed copies plus constant borders (padding) is still ONE launch.
__device__ __forceinline__ void fill_block(const DevPiece &sp, char *dst) {
  const uint4 fill = fill_unit<16>(sp);
  if (sp.kind == kDevStrip) {
    const uint64_t item = (uint64_t)(blockIdx.x - sp.first_block) * kAffineThreads + threadIdx.x;
    if (item >= sp.n_items) return;
    uint32_t rem = (uint32_t)item, strip = 0;
    int64_t dof = sp.doff;
    for (int k = sp.n_loops - 1; k >= 0; --k) {
      const uint32_t q = fast_div(rem, sp.fd[k]);
      const uint32_t i = rem - q * sp.ext[k];
      rem = q;
      dof += (int64_t)i * sp.dstride[k];
      if (k == sp.ku) strip = i;
    }
    const uint32_t left = sp.ku_ext - strip * kStrip;
#pragma unroll
    for (int u = 0; u < kStrip; ++u)
      if ((uint32_t)u < left) store_unit<16>(dst + dof + (int64_t)u * sp.ku_ds, fill);
  } else {
    const uint64_t item0 = (uint64_t)(blockIdx.x - sp.first_block) * (uint64_t)(kAffineThreads * kStrip) + threadIdx.x;
#pragma unroll
    for (int u = 0; u < kStrip; ++u) {
      const uint64_t L = item0 + (uint64_t)u * kAffineThreads;
      if (L >= sp.n_items) continue;
      uint32_t rem = (uint32_t)L;
      int64_t dof = sp.doff;
      for (int k = sp.n_loops - 1; k >= 0; --k) {
        const uint32_t q = fast_div(rem, sp.fd[k]);
        dof += (int64_t)(rem - q * sp.ext[k]) * sp.dstride[k];
        rem = q;
      }
      store_unit<16>(dst + dof, fill);
    }
  }
}

// CA = 16-byte chunks of a per tile; the tile always holds 1024 chunks:
//    8   128 bytes of a by 128 elements of b, the general shape;
//    4   64 bytes of a by 256 elements of b, for pieces or remainders at most 64 bytes long in a;
//   16   256 bytes of a by 64 elements of b, and
//   32   512 bytes of a by 32 elements of b, for pieces that short in b (NHWC -> NCHW with 64 or 32 channels);
//        rows must stay at least 128 bytes long for the swizzle, so 16 needs ES >= 2 and 32 needs ES >= 4.
// Either way a short extent no longer leaves the tile half empty.  The planner may also shorten the step along b
// (sp.step_b) so that the tiles of a row are evenly filled.
template <int ES, typename OffT, int CA>
__device__ __forceinline__ void transpose_tile(const DevPiece &sp, const PtrTable &ptrs, unsigned char *tile) {
  constexpr int EPU = 16 / ES;     // elements per 16-byte chunk
  constexpr int TA = CA * EPU;     // rows of the tile
  constexpr int TB = kTileB * 8 / CA;    // elements of b a tile can hold
  constexpr int RB = TB * ES;      // bytes per row
  constexpr int CB = RB / 16;      // chunks per row
  constexpr int G = CA >= 8 ? CA / 8 : 1;  // phase 2 walks a in groups of 8 chunks (one 128-byte line per row of lanes)
  constexpr int U = TA * CB / kTransposeThreads;
  static_assert(TA * RB == kTileBytes && U * kTransposeThreads == TA * CB && RB >= 128, "tile geometry");
  // phase 2: which chunk of a and which b (ES == 2: which pair of b) work item idx takes.  The 8 lanes that share a
  // b take 8 consecutive chunks of a (a full line of the destination), the 4 groups of 8 lanes 4 consecutive b.
  auto phase2_item = [](int idx, int *ca, int *bq) {
    if constexpr (CA >= 8) {
      const int lane = idx & 31, w = idx >> 5;
      *ca = (lane & 7) + 8 * (w % G);
      *bq = (lane >> 3) + 4 * (w / G);
    } else {
      *ca = idx % CA;
      *bq = idx / CA;
    }
  };

  const uint32_t step_b = sp.step_b;
  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_b);
  const uint32_t b0 = (t - q * sp.tiles_b) * step_b;
  t = q;
  q = fast_div(t, sp.fd_tiles_a);
  const uint32_t a0 = (t - q * sp.tiles_a) * TA;
  t = q;
  // Offsets are kept relative to the TENSORS' first bytes: with 32-bit OffT the arithmetic wraps around, which is
  // exact as long as the final offset fits 32 bits -- it does (the planner checks), whatever the signs of the
  // strides on the way.
  OffT sbase = (OffT)sp.soff, dbase = (OffT)sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (OffT)i * (OffT)sp.sstride[k];
    dbase += (OffT)i * (OffT)sp.dstride[k];
  }
  const char *src = ptrs.src[sp.input];
  char *dst = ptrs.dst(sp.out);
  const uint32_t ext_a = sp.ext_a;
  const uint32_t end_b = min(sp.ext_b, b0 + step_b);  // the tile's own end along b
  const FastDiv fa = sp.fd_a_in, fb = sp.fd_b_in;
  const bool split = fa.d < ext_a;       // a merges two loops
  const bool split_b = fb.d < sp.ext_b;  // b merges two loops
  const OffT sa0 = (OffT)sp.sa[0], sa1 = (OffT)sp.sa[1], db0 = (OffT)sp.db[0], db1 = (OffT)sp.db[1];
  // While the kernel before this one on the stream drains, ask L2 for this tile's source rows (a hint: it
  // reads nothing into the SM and is harmless whatever that kernel still writes); the loads after the wait
  // then start from L2 instead of paying a DRAM round trip with the memory system idle.  One bulk prefetch per
  // row; the instruction is issued lane by lane (some 500 instructions for the 64 rows), which is free here: the
  // block has nothing else to do until the wait returns.
  auto prefetch_rows_bulk = [&](OffT base, uint32_t pa0, uint32_t pb0) {
    const uint32_t a = pa0 + threadIdx.x;
    if (threadIdx.x < TA && a < ext_a && pb0 < sp.ext_b) {
      const uint32_t a_hi = fast_div(a, fa);
      const OffT off = base + (OffT)(a - a_hi * fa.d) * sa0 + (OffT)a_hi * sa1 + (OffT)(pb0 * ES);
      const uint32_t bytes = min(step_b, sp.ext_b - pb0) * ES;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src + off), "r"(bytes) : "memory");
    }
  };
  // The same hint line by line with the per-thread prefetch instruction (one warp instruction covers 32 lines; a
  // tile is 128 lines of 128 bytes: thread i < 128 asks for line i % LPR of row i / LPR): used between the loads and
  // the shared-memory stores, where instructions are not free.
  auto prefetch_rows = [&](OffT base, uint32_t pa0, uint32_t pb0) {
    constexpr int LPR = RB / 128;  // lines per tile row
    const uint32_t a = pa0 + threadIdx.x / LPR, line = threadIdx.x % LPR;
    if (threadIdx.x < TA * LPR && a < ext_a && pb0 < sp.ext_b) {
      const uint32_t bytes = min(step_b, sp.ext_b - pb0) * ES;
      if (line * 128 < bytes) {
        const uint32_t a_hi = fast_div(a, fa);
        const OffT off = base + (OffT)(a - a_hi * fa.d) * sa0 + (OffT)a_hi * sa1 + (OffT)(pb0 * ES);
        const char *row = src + off;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(row + line * 128));
        // a row that does not start on a line boundary ends in one line more
        if ((line + 1) * 128 >= bytes) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + bytes - 1));
      }
    }
  };
  // The same hint for the tile of the block that will take this block's place once it retires (`prefetch`
  // blocks further on in the grid): its loads will find their lines in L2.  Only within this piece: on a
  // launch of several small pieces (measured on configuration 4) hints for another piece's tiles cost more
  // than they save.
  auto prefetch_ahead = [&]() {
    if (sp.prefetch > 1 && threadIdx.x < 128) {
      uint32_t t2 = blockIdx.x - sp.first_block + (uint32_t)sp.prefetch;
      if (t2 < sp.n_blocks) {
        uint32_t q2 = fast_div(t2, sp.fd_tiles_b);
        const uint32_t nb0 = (t2 - q2 * sp.tiles_b) * step_b;
        t2 = q2;
        q2 = fast_div(t2, sp.fd_tiles_a);
        const uint32_t na0 = (t2 - q2 * sp.tiles_a) * TA;
        t2 = q2;
        OffT nbase = (OffT)sp.soff;
        for (int k = sp.n_loops - 1; k >= 0; --k) {
          q2 = fast_div(t2, sp.fd[k]);
          nbase += (OffT)(t2 - q2 * sp.ext[k]) * (OffT)sp.sstride[k];
          t2 = q2;
        }
        prefetch_rows(nbase, na0, nb0);
      }
    }
  };
  if (sp.prefetch) prefetch_rows_bulk(sbase, a0, b0);
  pdl_wait();

  // The common case -- the general tile shape, 2- or 4-byte elements, no merged indices, all rows of the tile inside
  // the piece -- with every address formed once per thread and stepped by constants: a third of the instructions
  // of the general path below.  (These kernels run against the power limit: instructions not issued are clock
  // kept.)  Block-uniform.
  if constexpr (CA == 8 && (ES == 2 || ES == 4)) {
    if (!split && !split_b && a0 + TA <= ext_a) {
      constexpr int RPU = kTransposeThreads / CB;  // tile rows between a thread's loads
      const int a_l0 = threadIdx.x / CB, cb = threadIdx.x % CB;
      const bool in_b = b0 + cb * EPU < end_b;
      const OffT first = sbase + (OffT)(a0 + a_l0) * sa0 + (OffT)((b0 + cb * EPU) * ES);
      const OffT step = (OffT)RPU * sa0;
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        v[u] = make_uint4(0, 0, 0, 0);
        if (in_b) v[u] = load_16(src + (OffT)(first + (OffT)u * step));
      }
      issue_barrier();  // all loads of the tile are in flight before the first shared-memory store waits for one
      prefetch_ahead();
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int a_l = a_l0 + u * RPU;
        *reinterpret_cast<uint4 *>(tile + a_l * RB + ((cb ^ ((a_l / EPU) & 7)) << 4)) = v[u];
      }
      __syncthreads();
      // phase 2.  Work item idx = thread + 256 u takes chunk ca of a and column (pair) bq + 32 u; 32 columns (pairs)
      // further on the tile's swizzle repeats, so the shared-memory address moves by a constant 128 bytes (ES = 2:
      // 64 columns) and the destination by a constant number of rows.
      const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
      const int ca = lane & 7, bq = (lane >> 3) + 4 * w;
      constexpr int COLS = ES == 2 ? 2 : 1;       // columns a work item stores
      constexpr int ROUNDS = ES == 2 ? U / 2 : U;
      const int b_l0 = bq * COLS;
      const unsigned char *p = tile + (ca * EPU) * RB + (((b_l0 / EPU) ^ ca) << 4) + (b_l0 % EPU) * ES;
      const OffT dfirst = dbase + (OffT)((a0 + ca * EPU) * ES) + (OffT)(b0 + b_l0) * db0;
      const OffT dstep = (OffT)(32 * COLS) * db0;
#pragma unroll
      for (int u = 0; u < ROUNDS; ++u) {
        const uint32_t b = b0 + b_l0 + u * 32 * COLS;
        if (b >= end_b) continue;  // extents and steps are even: with ES == 2, b + 1 is inside too
        const unsigned char *pu = p + u * 128;
        char *d = dst + (OffT)(dfirst + (OffT)u * dstep);
        if constexpr (ES == 2) {
          uint32_t r[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) r[j] = *reinterpret_cast<const uint32_t *>(pu + j * RB);
          uint4 lo, hi;
          lo.x = __byte_perm(r[0], r[1], 0x5410); hi.x = __byte_perm(r[0], r[1], 0x7632);
          lo.y = __byte_perm(r[2], r[3], 0x5410); hi.y = __byte_perm(r[2], r[3], 0x7632);
          lo.z = __byte_perm(r[4], r[5], 0x5410); hi.z = __byte_perm(r[4], r[5], 0x7632);
          lo.w = __byte_perm(r[6], r[7], 0x5410); hi.w = __byte_perm(r[6], r[7], 0x7632);
          __stcs(reinterpret_cast<uint4 *>(d), lo);
          __stcs(reinterpret_cast<uint4 *>(dst + (OffT)(dfirst + (OffT)u * dstep + db0)), hi);
        } else {
          uint4 out;
          out.x = *reinterpret_cast<const uint32_t *>(pu);
          out.y = *reinterpret_cast<const uint32_t *>(pu + RB);
          out.z = *reinterpret_cast<const uint32_t *>(pu + 2 * RB);
          out.w = *reinterpret_cast<const uint32_t *>(pu + 3 * RB);
          __stcs(reinterpret_cast<uint4 *>(d), out);
        }
      }
      return;
    }
  }

  // phase 1: global -> shared, 16 bytes along b
  uint4 v[U];
  {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = threadIdx.x + u * kTransposeThreads;
      const int a_l = idx / CB, cb = idx % CB;
      const uint32_t a = a0 + a_l, b = b0 + cb * EPU;
      v[u] = make_uint4(0, 0, 0, 0);
      if (a < ext_a && b < end_b) {
        OffT off = sbase + (OffT)(b * ES);
        if (split) {
          const uint32_t a_hi = fast_div(a, fa);
          off += (OffT)(a - a_hi * fa.d) * sa0 + (OffT)a_hi * sa1;
        } else {
          off += (OffT)a * sa0;
        }
        v[u] = load_16(src + off);
      }
    }
    issue_barrier();  // all loads of the tile are in flight before the first shared-memory store waits for one
    prefetch_ahead();
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = threadIdx.x + u * kTransposeThreads;
      const int a_l = idx / CB, cb = idx % CB;
      *reinterpret_cast<uint4 *>(tile + a_l * RB + ((cb ^ tile_swizzle<CA>(a_l / EPU)) << 4)) = v[u];
    }
  }
  __syncthreads();
  // phase 2: shared -> global, 16 bytes along a
  auto dst_of = [&](uint32_t a, uint32_t b) -> char * {
    OffT off = dbase + (OffT)(a * ES);
    if (split_b) {
      const uint32_t b_hi = fast_div(b, fb);
      off += (OffT)(b - b_hi * fb.d) * db0 + (OffT)b_hi * db1;
    } else {
      off += (OffT)b * db0;
    }
    return dst + off;
  };
  if constexpr (ES == 2) {
    // a thread takes two neighbouring b: the 8 words it reads hold both, so half as many shared loads
#pragma unroll
    for (int u = 0; u < U / 2; ++u) {
      const int idx = threadIdx.x + u * kTransposeThreads;
      int ca, b_l;
      phase2_item(idx, &ca, &b_l);
      b_l *= 2;
      const uint32_t a = a0 + ca * EPU, b = b0 + b_l;
      if (a < ext_a && b < end_b) {  // extents and steps are even: b + 1 is inside too
        const unsigned char *p = tile + (ca * EPU) * RB + (((b_l / EPU) ^ tile_swizzle<CA>(ca)) << 4) + (b_l % EPU) * ES;
        uint32_t r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) r[j] = *reinterpret_cast<const uint32_t *>(p + j * RB);
        uint4 lo, hi;
        lo.x = __byte_perm(r[0], r[1], 0x5410); hi.x = __byte_perm(r[0], r[1], 0x7632);
        lo.y = __byte_perm(r[2], r[3], 0x5410); hi.y = __byte_perm(r[2], r[3], 0x7632);
        lo.z = __byte_perm(r[4], r[5], 0x5410); hi.z = __byte_perm(r[4], r[5], 0x7632);
        lo.w = __byte_perm(r[6], r[7], 0x5410); hi.w = __byte_perm(r[6], r[7], 0x7632);
        __stcs(reinterpret_cast<uint4 *>(dst_of(a, b)), lo);
        __stcs(reinterpret_cast<uint4 *>(dst_of(a, b + 1)), hi);
      }
    }
  } else {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int idx = threadIdx.x + u * kTransposeThreads;
      int ca, b_l;
      phase2_item(idx, &ca, &b_l);
      const uint32_t a = a0 + ca * EPU, b = b0 + b_l;
      if (a < ext_a && b < end_b) __stcs(reinterpret_cast<uint4 *>(dst_of(a, b)), gather_column<ES, CA>(tile, ca, b_l));
    }
  }
}

template <int ES, typename OffT>
__device__ __forceinline__ void transpose_body(const DevPiece &sp, const PtrTable &ptrs) {
  __shared__ __align__(128) unsigned char tile[kTileBytes];
  if (sp.kind != kDevTranspose) {  // block-uniform
    pdl_wait();
    fill_block(sp, ptrs.dst(sp.out));
    return;
  }
  if (sp.tile_ca == 4) {
    transpose_tile<ES, OffT, 4>(sp, ptrs, tile);
    return;
  }
  if constexpr (ES >= 2) {
    if (sp.tile_ca == 16) {
      transpose_tile<ES, OffT, 16>(sp, ptrs, tile);
      return;
    }
  }
  if constexpr (ES >= 4) {
    if (sp.tile_ca == 32) {
      transpose_tile<ES, OffT, 32>(sp, ptrs, tile);
      return;
    }
  }
  transpose_tile<ES, OffT, 8>(sp, ptrs, tile);
}

// ---------------------------------------------------------------------------
// The same tiled transpose for pieces that are only aligned to UB < 16 bytes
// (extents that are multiples of UB/ES but not of 16/ES, e.g. 14x14 or 7x7
// feature maps): the tile, its shared-memory layout and the swizzle are
// unchanged, only the global accesses shrink to UB bytes.  Loads are issued in
// groups of eight.  Far slower than the 16-byte kernel per byte, but both
// global sides stay coalesced, which the element-wise gather cannot offer.
// ---------------------------------------------------------------------------
template <int ES>
__device__ __forceinline__ int tile_offset(int row, int col_byte) {
  constexpr int RB = kTileB * ES;
  return row * RB + ((((col_byte >> 4) ^ ((row / (16 / ES)) & 7)) << 4) | (col_byte & 15));
}

template <int ES, int UB, typename OffT>
__device__ __forceinline__ void transpose_narrow_body(const DevPiece &sp, const PtrTable &ptrs) {
  static_assert(UB >= ES && UB < 16, "narrow units");
  constexpr int EPN = UB / ES;          // elements per unit
  constexpr int TA = 8 * (16 / ES);     // tile rows, as in the 16-byte kernel
  constexpr int RB = kTileB * ES;
  constexpr int CBU = RB / UB;          // units per row
  constexpr int NCA = TA / EPN;         // units per destination run
  constexpr int N = kTileBytes / UB;    // units per tile
  constexpr int G = 8;                  // loads in flight per thread
  using T = typename Unit<UB>::T;
  using E = typename Unit<ES>::T;
  __shared__ __align__(128) unsigned char tile[kTileBytes];

  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_b);
  const uint32_t b0 = (t - q * sp.tiles_b) * kTileB;
  t = q;
  q = fast_div(t, sp.fd_tiles_a);
  const uint32_t a0 = (t - q * sp.tiles_a) * TA;
  t = q;
  int64_t sbase = sp.soff, dbase = sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (int64_t)i * sp.sstride[k];
    dbase += (int64_t)i * sp.dstride[k];
  }
  // offsets relative to the tensors' first bytes: 32-bit wrap-around arithmetic is then exact whatever the signs of
  // the strides (the final offset fits 32 bits)
  const char *src = ptrs.src[sp.input];
  char *dst = ptrs.dst(sp.out);
  const OffT sb = (OffT)sbase, dbs = (OffT)dbase;
  const uint32_t ext_a = sp.ext_a, ext_b = sp.ext_b;
  const FastDiv fa = sp.fd_a_in, fb = sp.fd_b_in;
  const OffT sa0 = (OffT)sp.sa[0], sa1 = (OffT)sp.sa[1], db0 = (OffT)sp.db[0], db1 = (OffT)sp.db[1];
  pdl_wait();

  for (int base = 0; base < N; base += G * kTransposeThreads) {
    T v[G];
    bool ok[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const int idx = base + threadIdx.x + g * kTransposeThreads;
      const int a_l = idx / CBU, cu = idx % CBU;
      const uint32_t a = a0 + a_l, b = b0 + cu * EPN;
      ok[g] = a < ext_a && b < ext_b;
      if (ok[g]) {
        const uint32_t a_hi = fast_div(a, fa);
        v[g] = load_unit<UB>(src + (OffT)(sb + (OffT)(b * ES) + (OffT)(a - a_hi * fa.d) * sa0 + (OffT)a_hi * sa1));
      }
    }
    issue_barrier();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const int idx = base + threadIdx.x + g * kTransposeThreads;
      if (ok[g]) *reinterpret_cast<T *>(tile + tile_offset<ES>(idx / CBU, (idx % CBU) * UB)) = v[g];
    }
  }
  __syncthreads();
#pragma unroll 4
  for (int idx = threadIdx.x; idx < N; idx += kTransposeThreads) {
    const int ca = idx % NCA, b_l = idx / NCA;
    const uint32_t a = a0 + ca * EPN, b = b0 + b_l;
    if (a < ext_a && b < ext_b) {
      union {
        T v;
        E e[EPN];
      } pk;
#pragma unroll
      for (int j = 0; j < EPN; ++j) pk.e[j] = *reinterpret_cast<const E *>(tile + tile_offset<ES>(ca * EPN + j, b_l * ES));
      const uint32_t b_hi = fast_div(b, fb);
      store_unit<UB>(dst + (OffT)(dbs + (OffT)(a * ES) + (OffT)(b - b_hi * fb.d) * db0 + (OffT)b_hi * db1), pk.v);
    }
  }
}

// ---------------------------------------------------------------------------
// The tiled transpose for pieces whose DESTINATION rows are not 16-byte aligned
// but whose source rows are (NHWC -> NCHW with an odd H*W).  Phase 1 is the
// aligned kernel's, over a taller tile.  Phase 2 works on the destination's
// own 16-byte grid: in row b the aligned slots start at the elements
// a = head + k * EPU, head = the elements from the row's start to the next
// 16-byte boundary, and the tile at a0 owns the eight slots that START inside
// [a0, a0 + TA).  A slot that starts near the end of that range needs up to
// EPU - 1 source rows beyond it, so the tile loads TA + EPU rows.  A slot that
// straddles the END of row b continues with the first elements of row b + 1
// when the rows follow each other in memory; those come from EPU more "wrap"
// rows (source rows 0 .. EPU-1), which a tile that can hold a row's end loads
// as well, and from column b + 1.  Every store is then a whole aligned 16-byte
// slot, except where the neighbour column is not in the tile: the last column
// of a tile stores its part of the straddling slot element by element, and the
// tile at a0 = 0 does the same for the head of its first column (both do it for
// every column when the rows do not follow each other).
// ---------------------------------------------------------------------------
template <int ES>
__device__ __forceinline__ void transpose_shifted_body(const DevPiece &sp, const PtrTable &ptrs) {
  constexpr int EPU = 16 / ES;
  constexpr int TA = 8 * EPU;            // slot starts a tile owns: a0 .. a0 + TA - 1
  constexpr int ROWS = TA + 2 * EPU;     // + EPU rows beyond that range + EPU wrap rows
  constexpr int RB = kTileB * ES;        // bytes per shared-memory row
  constexpr int CB = RB / 16;
  constexpr int U = ROWS * CB / kTransposeThreads;
  static_assert(U * kTransposeThreads == ROWS * CB, "tile geometry");
  using E = typename Unit<ES>::T;
  union Slot {
    uint4 vec;
    E e[EPU];
  };
  __shared__ __align__(128) unsigned char tile[ROWS * RB];

  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_b);
  const uint32_t b0 = (t - q * sp.tiles_b) * kTileB;
  t = q;
  q = fast_div(t, sp.fd_tiles_a);
  const uint32_t a0 = (t - q * sp.tiles_a) * TA;
  t = q;
  int64_t sbase = sp.soff, dbase = sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (int64_t)i * sp.sstride[k];
    dbase += (int64_t)i * sp.dstride[k];
  }
  const char *src = ptrs.src[sp.input] + sbase;
  char *dst = ptrs.dst(sp.out);  // dbase stays a byte offset: the slots are aligned relative to the tensor's start
  const uint32_t ext_a = sp.ext_a;
  const uint32_t end_b = min(sp.ext_b, b0 + kTileB);
  const FastDiv fa = sp.fd_a_in, fb = sp.fd_b_in;
  const bool holds_row_end = a0 + TA + EPU > ext_a;  // this tile may own the slot that straddles the end of a row
  const bool rows_follow = sp.shift_wrap != 0;       // row b + 1 starts where row b ends
  pdl_wait();

  // phase 1: rows [a0, a0 + TA + EPU) of the source, then (wrap) rows [0, EPU); 16-byte chunks along b
  uint4 v[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int idx = threadIdx.x + u * kTransposeThreads;
    const int r = idx / CB, cb = idx % CB;
    const uint32_t a = r < TA + EPU ? a0 + r : (uint32_t)(r - (TA + EPU)), b = b0 + cb * EPU;
    const bool wanted = r < TA + EPU ? a < ext_a : (holds_row_end && rows_follow && a < ext_a);
    v[u] = make_uint4(0, 0, 0, 0);
    if (wanted && b < end_b) {
      const uint32_t a_hi = fast_div(a, fa);
      v[u] = load_16(src + (int64_t)(a - a_hi * fa.d) * sp.sa[0] + (int64_t)a_hi * sp.sa[1] + (int64_t)b * ES);
    }
  }
  issue_barrier();
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int idx = threadIdx.x + u * kTransposeThreads;
    const int r = idx / CB, cb = idx % CB;
    *reinterpret_cast<uint4 *>(tile + r * RB + ((cb ^ ((r / EPU) & 7)) << 4)) = v[u];
  }
  __syncthreads();

  auto element = [&](int r, int b_l) -> E {  // tile row r, column b_l
    const int col = b_l * ES;
    return *reinterpret_cast<const E *>(tile + r * RB + ((((col >> 4) ^ ((r / EPU) & 7)) << 4) | (col & 15)));
  };
  // a slot that straddles the end of its row: elements a .. of column b_l, then rows wrap0 .. of column b_l + 1 if
  // that column is in the tile (whole store), else only the row's own elements, one by one
  auto straddling_slot = [&](char *p, uint32_t a, int r, int b_l, int wrap0, bool next_col) {
    Slot out;
#pragma unroll
    for (int e = 0; e < EPU; ++e) {
      if (a + e < ext_a) out.e[e] = element(r + e, b_l);
      else if (next_col) out.e[e] = element(wrap0 + (int)(a + e - ext_a), b_l + 1);
    }
    if (next_col) {
      __stcs(reinterpret_cast<uint4 *>(p), out.vec);
    } else {
#pragma unroll
      for (int e = 0; e < EPU; ++e)
        if (a + e < ext_a) store_unit<ES>(p + e * ES, out.e[e]);
    }
  };

  // Short rows (a whole row fits the tile, rows follow each other): the tile's destination is ONE contiguous
  // range, rows b0 .. end_b - 1, and an item is one aligned slot of that range, wherever it falls in a row.
  if (sp.tiles_a == 1 && rows_follow && fa.d >= ext_a) {
    const int64_t D0 = dbase + (int64_t)b0 * sp.db[0];  // start of row b0
    const uint32_t head0 = (uint32_t)((16 - (int)(D0 & 15)) & 15) / ES;
    const uint32_t n_flat = (end_b - b0) * ext_a;  // elements of the range
    if (threadIdx.x == 0)  // the elements before the first slot: the tile before this one could not store them
      for (uint32_t f = 0; f < head0 && f < n_flat; ++f) store_unit<ES>(dst + D0 + (int64_t)f * ES, element((int)f, 0));
    for (uint32_t f = head0 + threadIdx.x * EPU; f < n_flat; f += kTransposeThreads * EPU) {
      const uint32_t b_l = fast_div(f, fa), a = f - b_l * ext_a;
      char *p = dst + D0 + (int64_t)f * ES;
      if (a + EPU <= ext_a) {
        // EPU consecutive tile rows from row a on: they cross into the next group of EPU rows (the next swizzle)
        // after EPU - a % EPU of them
        const int col = (int)b_l * ES, chunk = col >> 4, g = (int)a / EPU;
        const unsigned char *base = tile + (int)a * RB + (col & 15);
        const int off_lo = (chunk ^ (g & 7)) << 4, off_hi = (chunk ^ ((g + 1) & 7)) << 4;
        const int split = EPU - (int)a % EPU;
        Slot out;
#pragma unroll
        for (int e = 0; e < EPU; ++e) out.e[e] = *reinterpret_cast<const E *>(base + e * RB + (e < split ? off_lo : off_hi));
        __stcs(reinterpret_cast<uint4 *>(p), out.vec);
      } else {
        straddling_slot(p, a, (int)a, (int)b_l, 0, b0 + b_l + 1 < end_b);
      }
    }
    return;
  }

  // phase 2: one item = one destination slot: slot k (0..7) of column b_l.  The eight lanes that share a column
  // take its eight slots (128 contiguous bytes); the four columns of a warp are two apart, so that their
  // elements sit in different shared-memory words.
#pragma unroll 2
  for (int idx = threadIdx.x; idx < 8 * kTileB; idx += kTransposeThreads) {
    const int k = idx & 7, sel = idx >> 3;
    const int b_l = ((sel & 3) << 1) + ((sel >> 2) & 1) + ((sel >> 3) << 3);
    const uint32_t b = b0 + b_l;
    if (b >= end_b) continue;
    const uint32_t b_hi = fast_div(b, fb);
    const int64_t D = dbase + (int64_t)(b - b_hi * fb.d) * sp.db[0] + (int64_t)b_hi * sp.db[1];  // row start
    const uint32_t head = (uint32_t)((16 - (int)(D & 15)) & 15) / ES;  // elements before the row's first slot
    // the head of the row belongs to the slot that straddles the end of the row before; this tile stores it
    // only when that slot's owner cannot (its column is the first of this tile, or rows do not follow each other)
    if (k == 0 && a0 == 0 && head > 0 && !(rows_follow && b_l > 0)) {
      for (uint32_t a = 0; a < head && a < ext_a; ++a) store_unit<ES>(dst + D + (int64_t)a * ES, element((int)a, b_l));
    }
    const uint32_t a_s = a0 + head + (uint32_t)k * EPU;  // first element of the slot
    if (a_s >= ext_a) continue;
    char *p = dst + D + (int64_t)a_s * ES;
    if (a_s + EPU <= ext_a) {
      // the slot lies inside the row (nearly all do): EPU consecutive tile rows from row head + k * EPU on, which
      // cross into the next group of EPU rows (the next swizzle) after EPU - head of them
      const int col = b_l * ES, chunk = col >> 4;
      const unsigned char *base = tile + (int)(head + (uint32_t)k * EPU) * RB + (col & 15);
      const int off_lo = (chunk ^ (k & 7)) << 4, off_hi = (chunk ^ ((k + 1) & 7)) << 4;
      const int split = EPU - (int)head;
      Slot out;
#pragma unroll
      for (int e = 0; e < EPU; ++e) out.e[e] = *reinterpret_cast<const E *>(base + e * RB + (e < split ? off_lo : off_hi));
      __stcs(reinterpret_cast<uint4 *>(p), out.vec);
    } else {
      straddling_slot(p, a_s, (int)(a_s - a0), b_l, TA + EPU, rows_follow && b + 1 < end_b);
    }
  }
}

// ---------------------------------------------------------------------------
// The transpose for pieces whose destination rows follow each other in memory
// (NHWC -> NCHW: a row is the H*W pixels of one channel), whatever the rows'
// alignment.  A block takes ALL of a for step_b consecutive b, so that what it
// writes is ONE contiguous range of the destination; the range starts on a
// 16-byte boundary because step_b is a multiple of 16/ES.  Dynamic shared
// memory holds that range as it will lie in memory:
//   phase 1  16-byte loads along b (step_b * ES contiguous bytes per a),
//            scattered element by element into the rows of the image;
//   phase 2  a linear copy of the image, 16 bytes per thread: whole lines,
//            whatever the length of a row.
// The lanes that share one a are the first 2^tile_ca of a group (tile_ca holds
// the logarithm here).
// ---------------------------------------------------------------------------
template <int ES, int THREADS, bool PAIRED>
__device__ __forceinline__ void transpose_flat_body(const DevPiece &sp, const PtrTable &ptrs) {
  constexpr int EPU = 16 / ES;
  // loads a thread keeps in flight: four in 32 registers where eight blocks of 256 threads share an SM; eight where
  // the panel's size leaves room for two to four blocks of 512 threads anyway
  constexpr int U = THREADS == 256 ? 4 : 8;
  using E = typename Unit<ES>::T;
  extern __shared__ __align__(128) unsigned char panel[];

  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_b);
  const uint32_t b0 = (t - q * sp.tiles_b) * sp.step_b;
  t = q;
  int64_t sbase = sp.soff, dbase = sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (int64_t)i * sp.sstride[k];
    dbase += (int64_t)i * sp.dstride[k];
  }
  const uint32_t ext_a = sp.ext_a, nb = min(sp.step_b, sp.ext_b - b0);
  const uint32_t row_bytes = ext_a * ES;
  const int lg = sp.tile_ca;
  const uint32_t cb = threadIdx.x & ((1u << lg) - 1u), a_step = THREADS >> lg;
  const bool lane_on = cb * EPU < nb;
  const FastDiv fa = sp.fd_a_in;
  const bool merged = fa.d < ext_a;
  const char *src = ptrs.src[sp.input] + sbase + (int64_t)b0 * ES + (int64_t)cb * 16;
  char *dst = ptrs.dst(sp.out) + dbase + (int64_t)b0 * sp.db[0];
  unsigned char *column = panel + cb * EPU * row_bytes;  // where this lane's first element of a = 0 goes
  // An L2 hint for this block's own segments, one line per a from the lanes with cb = 0, ahead of the dependency
  // wait: free for the blocks that sit in that wait while the kernel before this one drains.
  if (sp.prefetch && cb == 0) {
    const uint32_t seg = nb * ES;
    for (uint32_t a = threadIdx.x >> lg; a < ext_a; a += a_step) {
      const char *p = src + (merged ? (int64_t)(a - fast_div(a, fa) * fa.d) * sp.sa[0] + (int64_t)fast_div(a, fa) * sp.sa[1]
                                    : (int64_t)a * sp.sa[0]);
      asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
      if (seg > 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + 128));
    }
  }
  pdl_wait();

  // rounds of equal length: ten loads are five and five, not eight and two
  const uint32_t per_thread = (ext_a + a_step - 1) / a_step, rounds = (per_thread + U - 1) / U;
  const int u_round = (int)((per_thread + rounds - 1) / rounds);
  auto source_offset = [&](uint32_t a) -> int64_t {
    if (merged) {
      const uint32_t a_hi = fast_div(a, fa);
      return (int64_t)(a - a_hi * fa.d) * sp.sa[0] + (int64_t)a_hi * sp.sa[1];
    }
    return (int64_t)a * sp.sa[0];
  };
  // 2-byte elements, rows an even number of elements long (so that every row of the image starts on a 4-byte
  // boundary): a thread takes PAIRS of neighbouring a and stores 32-bit words, half the shared-memory stores
  // (PAIRED: the launch's pieces all qualify; a kernel of its own, so that neither form carries the other's registers)
  if constexpr (PAIRED) {
    constexpr int UP = U / 2;
    const uint32_t n_pairs = ext_a >> 1;
    const uint32_t pairs_per_thread = (n_pairs + a_step - 1) / a_step, pair_rounds = (pairs_per_thread + UP - 1) / UP;
    const int up_round = (int)((pairs_per_thread + pair_rounds - 1) / pair_rounds);
    for (uint32_t q0 = threadIdx.x >> lg; lane_on && q0 < n_pairs; q0 += (uint32_t)up_round * a_step) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < UP; ++u) {
        const uint32_t pr = q0 + (uint32_t)u * a_step;
        if (u < up_round && pr < n_pairs) {
          v[2 * u] = load_16(src + source_offset(2 * pr));
          v[2 * u + 1] = load_16(src + source_offset(2 * pr + 1));
        }
      }
      issue_barrier();
#pragma unroll
      for (int u = 0; u < UP; ++u) {
        const uint32_t pr = q0 + (uint32_t)u * a_step;
        if (u < up_round && pr < n_pairs) {
          unsigned char *p = column + pr * 4;
          const uint32_t w0[4] = {v[2 * u].x, v[2 * u].y, v[2 * u].z, v[2 * u].w};
          const uint32_t w1[4] = {v[2 * u + 1].x, v[2 * u + 1].y, v[2 * u + 1].z, v[2 * u + 1].w};
#pragma unroll
          for (int e = 0; e < EPU; ++e) {
            *reinterpret_cast<uint32_t *>(p) = __byte_perm(w0[e >> 1], w1[e >> 1], (e & 1) ? 0x7632 : 0x5410);
            p += row_bytes;
          }
        }
      }
    }
  }
  for (uint32_t a0 = threadIdx.x >> lg; !PAIRED && lane_on && a0 < ext_a; a0 += (uint32_t)u_round * a_step) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t a = a0 + (uint32_t)u * a_step;
      if (u < u_round && a < ext_a) v[u] = load_16(src + source_offset(a));
    }
    issue_barrier();
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t a = a0 + (uint32_t)u * a_step;
      if (u < u_round && a < ext_a) {
        unsigned char *p = column + a * ES;
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int e = 0; e < EPU; ++e) {
          E x;
          if constexpr (ES == 4) x = w[e];
          else x = (E)((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu));
          *reinterpret_cast<E *>(p) = x;
          p += row_bytes;
        }
      }
    }
  }
  __syncthreads();
  const uint32_t n16 = nb / EPU * ext_a;  // nb is a multiple of EPU: the range is a whole number of 16-byte units
#pragma unroll 4
  for (uint32_t i = threadIdx.x; i < n16; i += THREADS)
    __stcs(reinterpret_cast<uint4 *>(dst) + i, reinterpret_cast<const uint4 *>(panel)[i]);
}

// ---------------------------------------------------------------------------
// The mirror image: pieces whose SOURCE rows follow each other in memory
// (NCHW -> NHWC: a row is the H*W pixels of one channel), whatever the rows'
// alignment.  A block takes ALL of b for step_b consecutive a (the descriptor's
// step_b counts elements of a here), so that what it reads is ONE contiguous,
// 16-byte aligned range of the source:
//   phase 1  a linear copy of that range into shared memory;
//   phase 2  per b, the 16/ES elements of consecutive a are gathered from the
//            rows of the image, packed and stored as 16 bytes along a
//            (step_b * ES contiguous bytes of the destination per b).
// ---------------------------------------------------------------------------
template <int ES, int THREADS>
__device__ __forceinline__ void transpose_flat_source_body(const DevPiece &sp, const PtrTable &ptrs) {
  constexpr int EPU = 16 / ES;
  constexpr int U = THREADS == 256 ? 4 : 8;
  using E = typename Unit<ES>::T;
  extern __shared__ __align__(128) unsigned char panel[];

  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_a);
  const uint32_t a0 = (t - q * sp.tiles_a) * sp.step_b;
  t = q;
  int64_t sbase = sp.soff, dbase = sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (int64_t)i * sp.sstride[k];
    dbase += (int64_t)i * sp.dstride[k];
  }
  const uint32_t ext_b = sp.ext_b, na = min(sp.step_b, sp.ext_a - a0);
  const uint32_t row_bytes = ext_b * ES;
  const char *src = ptrs.src[sp.input] + sbase + (int64_t)a0 * sp.sa[0];
  // L2 hints (they read nothing into the SM): this block's panel while the kernel before this one drains, and,
  // once this block's first loads are out, the panel of the block that will take its place (`prefetch` blocks on).
  // A panel is one aligned range: one bulk prefetch from one thread.
  if (sp.prefetch && threadIdx.x == 0)
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(na * row_bytes) : "memory");
  pdl_wait();

  const uint32_t n16 = na / EPU * ext_b;  // na is a multiple of EPU: the range is a whole number of 16-byte units
  for (uint32_t i0 = threadIdx.x; i0 < n16; i0 += U * THREADS) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (i0 + u * THREADS < n16) v[u] = load_16(src + (size_t)(i0 + u * THREADS) * 16);
    if (i0 == 0 && sp.prefetch > 1) {  // thread 0, first round
      uint32_t t2 = blockIdx.x - sp.first_block + (uint32_t)sp.prefetch;
      if (t2 < sp.n_blocks) {
        uint32_t q2 = fast_div(t2, sp.fd_tiles_a);
        const uint32_t na0 = (t2 - q2 * sp.tiles_a) * sp.step_b;
        t2 = q2;
        int64_t nbase = sp.soff + (int64_t)na0 * sp.sa[0];
        for (int k = sp.n_loops - 1; k >= 0; --k) {
          q2 = fast_div(t2, sp.fd[k]);
          nbase += (int64_t)(t2 - q2 * sp.ext[k]) * sp.sstride[k];
          t2 = q2;
        }
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ptrs.src[sp.input] + nbase),
                     "r"(min(sp.step_b, sp.ext_a - na0) * row_bytes)
                     : "memory");
      }
    }
    issue_barrier();
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (i0 + u * THREADS < n16) reinterpret_cast<uint4 *>(panel)[i0 + u * THREADS] = v[u];
  }
  __syncthreads();

  const int lg = sp.tile_ca;
  const uint32_t ca = threadIdx.x & ((1u << lg) - 1u), b_step = THREADS >> lg;
  const bool lane_on = ca * EPU < na;
  const FastDiv fb = sp.fd_b_in;
  const bool merged = fb.d < ext_b;
  char *dst = ptrs.dst(sp.out) + dbase + (int64_t)a0 * ES + (int64_t)ca * 16;
  const unsigned char *column = panel + ca * EPU * row_bytes;  // this lane's first row of the image
  auto dest_offset = [&](uint32_t b) -> int64_t {
    if (merged) {
      const uint32_t b_hi = fast_div(b, fb);
      return (int64_t)(b - b_hi * fb.d) * sp.db[0] + (int64_t)b_hi * sp.db[1];
    }
    return (int64_t)b * sp.db[0];
  };
  // 2-byte elements, rows an even number of elements long: a thread takes PAIRS of neighbouring b, reads 32-bit
  // words (one per a, both b) and stores two vectors: half the shared-memory loads
  bool paired = false;
  if constexpr (ES == 2) paired = (ext_b & 1u) == 0;
  if (paired) {
#pragma unroll 2
    for (uint32_t pr = threadIdx.x >> lg; lane_on && pr < (ext_b >> 1); pr += b_step) {
      const unsigned char *p = column + pr * 4;
      uint32_t r[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) r[e] = *reinterpret_cast<const uint32_t *>(p + e * row_bytes);
      uint4 lo, hi;
      lo.x = __byte_perm(r[0], r[1], 0x5410); hi.x = __byte_perm(r[0], r[1], 0x7632);
      lo.y = __byte_perm(r[2], r[3], 0x5410); hi.y = __byte_perm(r[2], r[3], 0x7632);
      lo.z = __byte_perm(r[4], r[5], 0x5410); hi.z = __byte_perm(r[4], r[5], 0x7632);
      lo.w = __byte_perm(r[6], r[7], 0x5410); hi.w = __byte_perm(r[6], r[7], 0x7632);
      __stcs(reinterpret_cast<uint4 *>(dst + dest_offset(2 * pr)), lo);
      __stcs(reinterpret_cast<uint4 *>(dst + dest_offset(2 * pr + 1)), hi);
    }
    return;
  }
#pragma unroll 2
  for (uint32_t b = threadIdx.x >> lg; lane_on && b < ext_b; b += b_step) {
    const unsigned char *p = column + b * ES;
    uint32_t w[4];
    if constexpr (ES == 4) {
#pragma unroll
      for (int e = 0; e < 4; ++e) w[e] = *reinterpret_cast<const uint32_t *>(p + e * row_bytes);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t lo = *reinterpret_cast<const uint16_t *>(p + (2 * e) * row_bytes);
        const uint32_t hi = *reinterpret_cast<const uint16_t *>(p + (2 * e + 1) * row_bytes);
        w[e] = lo | (hi << 16);
      }
    }
    __stcs(reinterpret_cast<uint4 *>(dst + dest_offset(b)), make_uint4(w[0], w[1], w[2], w[3]));
  }
}

// ---------------------------------------------------------------------------
// The tiled transpose for pieces whose SOURCE rows are not 16-byte aligned but
// whose destination rows are (NCHW -> NHWC with an odd H*W: 7x7, 35x35, 55x55
// maps).  Phase 1 still loads aligned 16-byte chunks: the 16 lanes that share a
// row load the chunks that cover its bytes, then every lane builds the
// UN-shifted chunk (row bytes [16k + s, 16k + 16 + s), s = row address mod 16)
// from its own four words and its neighbour's (one shuffle per word, a
// two-stage word select and a funnel shift) and stores it where the aligned
// kernel would have.  Phase 2 is the aligned kernel's.  Tile: 128 bytes of a by
// 14 chunks of b, so that a shifted row needs at most 15 aligned chunks.
// ---------------------------------------------------------------------------
template <int ES>
__device__ __forceinline__ void transpose_realign_body(const DevPiece &sp, const PtrTable &ptrs) {
  constexpr int EPU = 16 / ES;
  constexpr int TA = 8 * EPU;      // rows
  constexpr int TBR = 14 * EPU;    // elements of b per tile
  constexpr int PITCH = 256;       // bytes per shared-memory row (16 chunks)
  constexpr int PASSES = TA / 16;  // 16 rows per pass: 16 lanes per row
  __shared__ __align__(128) unsigned char tile[TA * PITCH];

  uint32_t t = blockIdx.x - sp.first_block;
  uint32_t q = fast_div(t, sp.fd_tiles_b);
  const uint32_t b0 = (t - q * sp.tiles_b) * TBR;
  t = q;
  q = fast_div(t, sp.fd_tiles_a);
  const uint32_t a0 = (t - q * sp.tiles_a) * TA;
  t = q;
  int64_t sbase = sp.soff, dbase = sp.doff;
  for (int k = sp.n_loops - 1; k >= 0; --k) {
    q = fast_div(t, sp.fd[k]);
    const uint32_t i = t - q * sp.ext[k];
    t = q;
    sbase += (int64_t)i * sp.sstride[k];
    dbase += (int64_t)i * sp.dstride[k];
  }
  const char *src = ptrs.src[sp.input];
  char *dst = ptrs.dst(sp.out) + dbase;
  const uint32_t ext_a = sp.ext_a, ext_b = sp.ext_b;
  const FastDiv fa = sp.fd_a_in, fb = sp.fd_b_in;
  const int nb = (int)min((uint32_t)TBR, ext_b - b0);
  const int k = threadIdx.x & 15;  // chunk of the row this lane loads and, un-shifted, stores
  pdl_wait();

  uint4 v[PASSES];
  int shift[PASSES];
#pragma unroll
  for (int u = 0; u < PASSES; ++u) {
    const int a_l = (threadIdx.x >> 4) + 16 * u;
    const uint32_t a = a0 + a_l;
    v[u] = make_uint4(0, 0, 0, 0);
    shift[u] = 0;
    if (a < ext_a) {
      const uint32_t a_hi = fast_div(a, fa);
      const int64_t g = sbase + (int64_t)(a - a_hi * fa.d) * sp.sa[0] + (int64_t)a_hi * sp.sa[1] + (int64_t)b0 * ES;
      shift[u] = (int)(g & 15);
      const int64_t addr = (g & ~(int64_t)15) + 16 * k;
      if (addr < g + (int64_t)nb * ES) {  // the chunk overlaps the row's bytes
        if (addr + 16 <= sp.src_bytes) {
          v[u] = load_16(src + addr);
        } else {  // the tensor ends inside this chunk
          union {
            uint4 w;
            typename Unit<ES>::T e[EPU];
          } pk;
          pk.w = make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int e = 0; e < EPU; ++e)
            if (addr + (e + 1) * ES <= sp.src_bytes) pk.e[e] = load_unit<ES>(src + addr + e * ES);
          v[u] = pk.w;
        }
      }
    }
  }
  issue_barrier();
#pragma unroll
  for (int u = 0; u < PASSES; ++u) {
    const int a_l = (threadIdx.x >> 4) + 16 * u;
    // the neighbour's chunk (lane k + 1 of the same 16-lane row group); every lane takes part
    uint32_t w[8] = {v[u].x, v[u].y, v[u].z, v[u].w, 0, 0, 0, 0};
    w[4] = __shfl_down_sync(0xFFFFFFFFu, v[u].x, 1, 16);
    w[5] = __shfl_down_sync(0xFFFFFFFFu, v[u].y, 1, 16);
    w[6] = __shfl_down_sync(0xFFFFFFFFu, v[u].z, 1, 16);
    w[7] = __shfl_down_sync(0xFFFFFFFFu, v[u].w, 1, 16);
    const int o = shift[u] >> 2, bits = (shift[u] & 3) * 8;
    uint32_t x[6], y[5];
#pragma unroll
    for (int i = 0; i < 6; ++i) x[i] = (o & 2) ? w[i + 2] : w[i];
#pragma unroll
    for (int i = 0; i < 5; ++i) y[i] = (o & 1) ? x[i + 1] : x[i];
    uint4 out;
    out.x = __funnelshift_r(y[0], y[1], bits);
    out.y = __funnelshift_r(y[1], y[2], bits);
    out.z = __funnelshift_r(y[2], y[3], bits);
    out.w = __funnelshift_r(y[3], y[4], bits);
    if (a0 + a_l < ext_a && k * EPU < nb)
      *reinterpret_cast<uint4 *>(tile + a_l * PITCH + ((k ^ ((a_l / EPU) & 7)) << 4)) = out;
  }
  __syncthreads();

  const bool split_b = fb.d < ext_b;
  auto dst_of = [&](uint32_t a, uint32_t b) -> char * {
    int64_t off = (int64_t)a * ES;
    if (split_b) {
      const uint32_t b_hi = fast_div(b, fb);
      off += (int64_t)(b - b_hi * fb.d) * sp.db[0] + (int64_t)b_hi * sp.db[1];
    } else {
      off += (int64_t)b * sp.db[0];
    }
    return dst + off;
  };
  if constexpr (ES == 2) {
#pragma unroll 2
    for (int idx = threadIdx.x; idx < (TBR / 2) * 8; idx += kTransposeThreads) {
      const int ca = idx & 7, b_l = (idx >> 3) * 2;
      const uint32_t a = a0 + ca * EPU, b = b0 + b_l;
      if (a < ext_a && b_l < nb) {
        const unsigned char *p = tile + (ca * EPU) * PITCH + (((b_l / EPU) ^ ca) << 4) + (b_l % EPU) * ES;
        uint32_t r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) r[j] = *reinterpret_cast<const uint32_t *>(p + j * PITCH);
        uint4 lo, hi;
        lo.x = __byte_perm(r[0], r[1], 0x5410); hi.x = __byte_perm(r[0], r[1], 0x7632);
        lo.y = __byte_perm(r[2], r[3], 0x5410); hi.y = __byte_perm(r[2], r[3], 0x7632);
        lo.z = __byte_perm(r[4], r[5], 0x5410); hi.z = __byte_perm(r[4], r[5], 0x7632);
        lo.w = __byte_perm(r[6], r[7], 0x5410); hi.w = __byte_perm(r[6], r[7], 0x7632);
        __stcs(reinterpret_cast<uint4 *>(dst_of(a, b)), lo);
        if (b_l + 1 < nb) __stcs(reinterpret_cast<uint4 *>(dst_of(a, b + 1)), hi);  // an odd extent ends on a lone b
      }
    }
  } else {
#pragma unroll 2
    for (int idx = threadIdx.x; idx < TBR * 8; idx += kTransposeThreads) {
      const int ca = idx & 7, b_l = idx >> 3;
      const uint32_t a = a0 + ca * EPU, b = b0 + b_l;
      if (a < ext_a && b_l < nb) {
        union {
          uint4 w;
          typename Unit<ES>::T e[EPU];
        } pk;
        const int col = b_l * ES;
#pragma unroll
        for (int j = 0; j < EPU; ++j)
          pk.e[j] = *reinterpret_cast<const typename Unit<ES>::T *>(tile + (ca * EPU + j) * PITCH + (((col >> 4) ^ ca) << 4) + (col & 15));
        __stcs(reinterpret_cast<uint4 *>(dst_of(a, b)), pk.w);
      }
    }
  }
}

// ---------------------------------------------------------------------------
// Entry kernels.  Each family has two: the *_param kernels get up to
// kParamPieces descriptors BY VALUE in the kernel parameters (constant bank: a
// block starts its index arithmetic without a round trip to global memory),
// the *_table kernels read them from a descriptor table in global memory
// (launches with more pieces, and amap_execute_static).
// ---------------------------------------------------------------------------
constexpr int kParamPieces = 16;
struct LaunchDesc {
  int32_t n_pieces;
  int32_t pad_;
  DevPiece piece[kParamPieces];
};

__device__ __forceinline__ const DevPiece &param_piece(const LaunchDesc &ld) {
  int p = 0;
  while (p + 1 < ld.n_pieces && blockIdx.x >= ld.piece[p + 1].first_block) ++p;
  return ld.piece[p];
}

template <int V, int U, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_affine_param(const __grid_constant__ LaunchDesc ld, PtrTable ptrs) {
  pdl_launch_dependents();
  affine_body<V, U, NC, OffT>(param_piece(ld), ptrs);
}
template <int V, int U, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_affine_table(const DevPiece *__restrict__ table, int first_piece,
                                                                     int n_pieces, PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  affine_body<V, U, NC, OffT>(sp, ptrs);
}

template <int V, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_strip_param(const __grid_constant__ LaunchDesc ld, PtrTable ptrs) {
  pdl_launch_dependents();
  strip_body<V, NC, OffT>(param_piece(ld), ptrs);
}
template <int V, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_strip_table(const DevPiece *__restrict__ table, int first_piece,
                                                                    int n_pieces, PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  strip_body<V, NC, OffT>(sp, ptrs);
}

template <int ES, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads, 8) amap_transpose_param(const __grid_constant__ LaunchDesc ld,
                                                                              PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_body<ES, OffT>(param_piece(ld), ptrs);
}
template <int ES, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_table(const DevPiece *__restrict__ table,
                                                                           int first_piece, int n_pieces, PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_body<ES, OffT>(sp, ptrs);
}

template <int ES, int UB, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_narrow_param(const __grid_constant__ LaunchDesc ld,
                                                                                  PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_narrow_body<ES, UB, OffT>(param_piece(ld), ptrs);
}
template <int ES, int UB, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_narrow_table(const DevPiece *__restrict__ table,
                                                                                  int first_piece, int n_pieces,
                                                                                  PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_narrow_body<ES, UB, OffT>(sp, ptrs);
}

template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_shifted_param(const __grid_constant__ LaunchDesc ld,
                                                                                   PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_shifted_body<ES>(param_piece(ld), ptrs);
}
template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_shifted_table(const DevPiece *__restrict__ table,
                                                                                   int first_piece, int n_pieces,
                                                                                   PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_shifted_body<ES>(sp, ptrs);
}

// Single-piece launches (the common case) pass just that descriptor: a ninth of the parameter bytes.
template <int V, int U, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_affine_one(const __grid_constant__ DevPiece p, PtrTable ptrs) {
  pdl_launch_dependents();
  affine_body<V, U, NC, OffT>(p, ptrs);
}
template <int V, int NC, typename OffT>
__global__ void __launch_bounds__(kAffineThreads) amap_strip_one(const __grid_constant__ DevPiece p, PtrTable ptrs) {
  pdl_launch_dependents();
  strip_body<V, NC, OffT>(p, ptrs);
}
template <int ES, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads, 8) amap_transpose_one(const __grid_constant__ DevPiece p, PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_body<ES, OffT>(p, ptrs);
}
template <int ES, int UB, typename OffT>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_narrow_one(const __grid_constant__ DevPiece p,
                                                                                PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_narrow_body<ES, UB, OffT>(p, ptrs);
}
template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_shifted_one(const __grid_constant__ DevPiece p,
                                                                                 PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_shifted_body<ES>(p, ptrs);
}

template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_realign_param(const __grid_constant__ LaunchDesc ld,
                                                                                   PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_realign_body<ES>(param_piece(ld), ptrs);
}
template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_realign_table(const DevPiece *__restrict__ table,
                                                                                   int first_piece, int n_pieces,
                                                                                   PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_realign_body<ES>(sp, ptrs);
}
template <int ES>
__global__ void __launch_bounds__(kTransposeThreads) amap_transpose_realign_one(const __grid_constant__ DevPiece p,
                                                                                 PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_realign_body<ES>(p, ptrs);
}

// The flat-destination transpose runs with the dynamic shared memory its launch asks for: small panels with eight
// blocks of 256 threads per SM (32 registers per thread), large ones with blocks of 512 threads (64 registers).
template <int ES, int THREADS, bool PAIRED>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2) amap_transpose_flat_param(const __grid_constant__ LaunchDesc ld,
                                                                                    PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_flat_body<ES, THREADS, PAIRED>(param_piece(ld), ptrs);
}
template <int ES, int THREADS, bool PAIRED>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2) amap_transpose_flat_table(const DevPiece *__restrict__ table,
                                                                                    int first_piece, int n_pieces,
                                                                                    PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_flat_body<ES, THREADS, PAIRED>(sp, ptrs);
}
template <int ES, int THREADS, bool PAIRED>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2) amap_transpose_flat_one(const __grid_constant__ DevPiece p,
                                                                                  PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_flat_body<ES, THREADS, PAIRED>(p, ptrs);
}

template <int ES, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2)
    amap_transpose_flat_source_param(const __grid_constant__ LaunchDesc ld, PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_flat_source_body<ES, THREADS>(param_piece(ld), ptrs);
}
template <int ES, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2)
    amap_transpose_flat_source_table(const DevPiece *__restrict__ table, int first_piece, int n_pieces, PtrTable ptrs) {
  __shared__ DevPiece sp;
  pdl_launch_dependents();
  fetch_piece(table, first_piece, n_pieces, &sp);
  transpose_flat_source_body<ES, THREADS>(sp, ptrs);
}
template <int ES, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? 8 : 2)
    amap_transpose_flat_source_one(const __grid_constant__ DevPiece p, PtrTable ptrs) {
  pdl_launch_dependents();
  transpose_flat_source_body<ES, THREADS>(p, ptrs);
}

}  // namespace amap
