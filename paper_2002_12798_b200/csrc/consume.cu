// A consumer that reads THROUGH a composed map (amap_device.h): the row sums of the chain's result, computed from the
// external inputs without the result ever being written.  This is the GPU reading of the paper's Section 2.2 (no
// copy between an operator and the next one that needs its data laid out differently): the composed access map g'
// of Section 2.1, equation (2), is evaluated inside the consuming kernel.
#include <cuda_runtime.h>

#include "amap.h"
#include "amap_device.h"

namespace {

constexpr int kMaxViewInputs = 24;
constexpr int kThreads = 256;

struct ViewPtrs {
  const char *src[kMaxViewInputs];
};

// sum of the 16 / ES unsigned elements held in 16 bytes
template <int ES>
__device__ __forceinline__ uint32_t vector_sum(uint4 v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  uint32_t acc = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if constexpr (ES == 4) acc += w[k];
    else if constexpr (ES == 2) acc += (w[k] & 0xFFFFu) + (w[k] >> 16);
    else acc += (w[k] & 0xFFu) + ((w[k] >> 8) & 0xFFu) + ((w[k] >> 16) & 0xFFu) + (w[k] >> 24);
  }
  return acc;
}

template <int ES>
__device__ __forceinline__ uint32_t element_at(const char *p) {
  if constexpr (ES == 4) return *reinterpret_cast<const uint32_t *>(p);
  else if constexpr (ES == 2) return *reinterpret_cast<const uint16_t *>(p);
  else return *reinterpret_cast<const uint8_t *>(p);
}

// A group of G lanes (a power of two, the whole warp for long rows) takes `rows_per_group` consecutive rows of the
// (virtual) result; a lane takes 16 bytes' worth of consecutive output elements at a time, asks the view where they
// come from, and fetches them with one vector load when they are one aligned run.  Four such loads are issued
// before the first is consumed, so that every lane keeps several requests in flight.
template <int ES>
__global__ void __launch_bounds__(kThreads) row_sums_kernel(const __grid_constant__ amap_device_view v, ViewPtrs ptrs,
                                                            int64_t rows, int64_t cols, uint32_t *__restrict__ sums,
                                                            int G, int rows_per_group) {
  constexpr int EPV = 16 / ES;
  constexpr int kBatch = 4;
  const int lane = threadIdx.x & 31, gl = lane & (G - 1);
  const int64_t group = ((int64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5)) * (32 / G) + lane / G;
  const uint32_t elem_mask = ES == 4 ? 0xFFFFFFFFu : ((1u << (8 * ES)) - 1u);
  const int64_t chunks = (cols + EPV - 1) / EPV;
  for (int u = 0; u < rows_per_group; ++u) {  // the same trip count for every lane: the shuffles below are warp-wide
    const int64_t row = group * rows_per_group + u;
    uint32_t acc = 0;
    for (int64_t t0 = 0; t0 < chunks; t0 += (int64_t)kBatch * G) {
      const char *p[kBatch];
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        p[j] = nullptr;
        const int64_t c = (t0 + gl + (int64_t)j * G) * EPV;
        if (row >= rows || c >= cols) continue;
        const int64_t o = row * cols + c;
        const int n = (int)(cols - c < EPV ? cols - c : EPV);
        amap_view_source s;
        if (amap_view_locate(v, o, &s) && s.run >= n) {
          if (s.input < 0) {
            acc += (uint32_t)n * ((uint32_t)s.fill_bits & elem_mask);
          } else {
            const char *q = ptrs.src[s.input] + s.index * ES;
            if (n == EPV && (reinterpret_cast<uintptr_t>(q) & 15) == 0) {
              p[j] = q;  // the common case: loaded below, together with the batch's other chunks
            } else {
              for (int e = 0; e < n; ++e) acc += element_at<ES>(q + e * ES);
            }
          }
        } else {  // the elements come from different places: one by one
          for (int e = 0; e < n; ++e) {
            if (!amap_view_locate(v, o + e, &s)) continue;
            acc += s.input < 0 ? ((uint32_t)s.fill_bits & elem_mask) : element_at<ES>(ptrs.src[s.input] + s.index * ES);
          }
        }
      }
      uint4 val[kBatch];
#pragma unroll
      for (int j = 0; j < kBatch; ++j)
        if (p[j]) val[j] = __ldg(reinterpret_cast<const uint4 *>(p[j]));
#pragma unroll
      for (int j = 0; j < kBatch; ++j)
        if (p[j]) acc += vector_sum<ES>(val[j]);
    }
    for (int d = G >> 1; d > 0; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if (gl == 0 && row < rows) sums[row] = acc;
  }
}

}  // namespace

extern "C" int amap_consume_row_sums(const amap_device_view *view, const void *const *src_dev_ptrs, int64_t rows,
                                     int64_t cols, uint32_t *sums_dev, void *cuda_stream) {
  if (!view || rows < 0 || cols < 0 || (rows > 0 && !sums_dev)) return AMAP_EINVAL;
  if (view->n_pieces < 0 || view->n_pieces > AMAP_VIEW_MAX_PIECES || view->n_inputs < 0 || view->n_inputs > kMaxViewInputs)
    return AMAP_EINVAL;
  if (view->elem_size != 1 && view->elem_size != 2 && view->elem_size != 4) return AMAP_EUNSUPPORTED;
  if (rows == 0) return AMAP_OK;
  if (cols == 0 || rows != view->out_numel / cols || rows * cols != view->out_numel) return AMAP_EINVAL;
  if (view->n_inputs > 0 && !src_dev_ptrs) return AMAP_EINVAL;
  ViewPtrs ptrs = {};
  for (int q = 0; q < view->n_inputs; ++q) {
    if (reinterpret_cast<uintptr_t>(src_dev_ptrs[q]) & 15) return AMAP_EALIGN;
    ptrs.src[q] = static_cast<const char *>(src_dev_ptrs[q]);
  }
  // lanes per row: the next power of two at or above the row's 16-byte chunks, at most a warp; short rows share a
  // warp, and a group takes several of them so that every lane has about four loads to issue
  const int64_t chunks = (cols * view->elem_size + 15) / 16;
  int G = 1;
  while (G < 32 && G < chunks) G <<= 1;
  const int per_lane = (int)((chunks + G - 1) / G);
  const int rows_per_group = per_lane >= 4 ? 1 : 4 / per_lane;
  const int64_t groups = (rows + rows_per_group - 1) / rows_per_group;
  const int64_t warps = (groups + 32 / G - 1) / (32 / G);
  const int64_t blocks = (warps + kThreads / 32 - 1) / (kThreads / 32);
  if (blocks > 0x7FFFFFFF) return AMAP_EOVERFLOW;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  switch (view->elem_size) {
    case 4: row_sums_kernel<4><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
    case 2: row_sums_kernel<2><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
    default: row_sums_kernel<1><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
  }
  return cudaGetLastError() == cudaSuccess ? AMAP_OK : AMAP_ECUDA;
}
