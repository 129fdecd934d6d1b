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

template <int V>
__device__ __forceinline__ typename Unit<V>::T load_unit(const char *p) {
  return __ldg(reinterpret_cast<const typename Unit<V>::T *>(p));
}

template <int V>
__device__ __forceinline__ void store_unit(char *p, typename Unit<V>::T v) {
  __stcs(reinterpret_cast<typename Unit<V>::T *>(p), v);
}

// find the piece a block belongs to and copy its descriptor to shared memory
__device__ __forceinline__ void fetch_piece(const DevPiece *__restrict__ table, int first_piece, int n_pieces,
                                            DevPiece *sp) {
  int p = first_piece;
  const int last = first_piece + n_pieces - 1;
  while (p < last && blockIdx.x >= table[p + 1].first_block) ++p;
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
// every piece, including non-injective loads (overlapping windows).  All U
// loads are issued before the first store so that each thread keeps U
// independent requests in flight.
// ---------------------------------------------------------------------------
constexpr int kAffineThreads = 256;

template <int V, int U>
__global__ void __launch_bounds__(kAffineThreads) amap_affine_kernel(const DevPiece *__restrict__ table, int first_piece,
                                                                      int n_pieces, PtrTable ptrs) {
  __shared__ DevPiece sp;
  fetch_piece(table, first_piece, n_pieces, &sp);
  using T = typename Unit<V>::T;
  const int n = sp.n_loops;
  const int n_cons = sp.n_guards + sp.n_domain;
  const uint64_t item0 = (uint64_t)(blockIdx.x - sp.first_block) * (uint64_t)(kAffineThreads * U) + threadIdx.x;
  const char *src = (sp.input >= 0) ? ptrs.src[sp.input] : nullptr;
  char *dst = ptrs.dst;

  int64_t so[U], doff[U];
  bool live[U], load[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const uint64_t L = item0 + (uint64_t)u * kAffineThreads;
    live[u] = L < sp.n_items;
    load[u] = live[u] && (src != nullptr);
    uint32_t rem = live[u] ? (uint32_t)L : 0u;
    int64_t s = sp.soff, d = sp.doff;
    int64_t acc[kDevMaxCons];
#pragma unroll
    for (int c = 0; c < kDevMaxCons; ++c) acc[c] = 0;
    for (int k = n - 1; k >= 0; --k) {
      const uint32_t q = fast_div(rem, sp.fd[k]);
      const uint32_t i = rem - q * sp.ext[k];
      rem = q;
      s += (int64_t)i * sp.sstride[k];
      d += (int64_t)i * sp.dstride[k];
      if (n_cons > 0) {
#pragma unroll
        for (int c = 0; c < kDevMaxCons; ++c)
          if (c < n_cons) acc[c] += (int64_t)sp.cons[c].coef[k] * (int64_t)i;
      }
    }
    if (n_cons > 0) {
#pragma unroll
      for (int c = 0; c < kDevMaxCons; ++c)
        if (c < n_cons) {
          const int64_t v = acc[c] + sp.cons[c].off;
          const bool ok = (v >= 0) && (v < sp.cons[c].extent);
          if (c < sp.n_guards) load[u] = load[u] && ok;   // a failed guard stores the fill value
          else live[u] = live[u] && ok;                    // outside the piece's domain: nothing to do
        }
    }
    so[u] = s;
    doff[u] = d;
  }
  T val[U];
  const T fill = fill_unit<V>(sp);
#pragma unroll
  for (int u = 0; u < U; ++u) val[u] = (load[u] && live[u]) ? load_unit<V>(src + so[u]) : fill;
#pragma unroll
  for (int u = 0; u < U; ++u)
    if (live[u]) store_unit<V>(dst + doff[u], val[u]);
}

}  // namespace amap
