// A consumer that reads THROUGH a composed map (amap_device.h): the row sums of the chain's result, computed from the
// external inputs without the result ever being written.  This is the GPU reading of the paper's Section 2.2 (no
// copy between an operator and the next one that needs its data laid out differently): the composed access map g'
// of Section 2.1, equation (2), is evaluated inside the consuming kernel.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstring>

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

// The same sums for views whose rows are whole runs of one piece each (amap_view_rows): the loops outside a row are
// decoded once per row, the runs inside it come from a table the block keeps in shared memory.  A group of G lanes
// takes a row; of every run a lane takes up to four 16-byte vectors (G apart), all loaded before the first is
// consumed.  Blocks stride over the rows.
template <int ES>
__global__ void __launch_bounds__(kThreads, 4) row_sums_by_runs_kernel(const __grid_constant__ amap_device_view v,
                                                                    const __grid_constant__ amap_view_rows rows_param,
                                                                    ViewPtrs ptrs, int64_t rows, uint32_t *__restrict__ sums,
                                                                    int G) {
  constexpr int EPV = 16 / ES;
  constexpr int kBatch = 4;
  __shared__ amap_view_rows R;
  {
    const uint32_t *src = reinterpret_cast<const uint32_t *>(&rows_param);
    uint32_t *dst = reinterpret_cast<uint32_t *>(&R);
    const int words = (int)((offsetof(amap_view_rows, piece) + (size_t)rows_param.n_pieces * sizeof(amap_view_row_piece)) / 4);
    for (int w = threadIdx.x; w < words; w += kThreads) dst[w] = src[w];
    __syncthreads();
  }
  const int lane = threadIdx.x & 31, gl = lane & (G - 1);
  const int64_t groups_per_block = kThreads / G;
  const uint32_t cols = R.cols;
  const uint32_t elem_mask = ES == 4 ? 0xFFFFFFFFu : ((1u << (8 * ES)) - 1u);
  // the same trip count for every lane of a warp: the shuffles below are warp-wide
  for (int64_t base = (int64_t)blockIdx.x * groups_per_block; base < rows; base += (int64_t)gridDim.x * groups_per_block) {
    const int64_t row = base + threadIdx.x / G;
    uint32_t acc = 0;
    amap_view_row_cursor cur;
    cur.piece = -1;
    if (row < rows) amap_view_row_seek(R, (uint32_t)(row * cols), &cur);
    if (cur.piece >= 0) {
      const amap_view_row_piece &rp = R.piece[cur.piece];
      const uint32_t run_len = (uint32_t)rp.run_len, fill = rp.fill_bits_lo & elem_mask;
      const bool vectors = (run_len * ES) % 16 == 0;
      const uint32_t n_vec = run_len / EPV;
      const char *in = rp.input >= 0 ? ptrs.src[rp.input] : nullptr;
      for (int j = 0; j < rp.n_runs; ++j) {
        uint32_t s;
        if (!amap_view_row_run(rp, cur, j, &s)) {
          if (gl == 0) acc += run_len * fill;
          continue;
        }
        const char *q = in + (size_t)s * ES;
        if (vectors && (reinterpret_cast<uintptr_t>(q) & 15) == 0) {  // the common case
          const uint4 *q16 = reinterpret_cast<const uint4 *>(q);
          uint4 val[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u)
            if ((uint32_t)(gl + u * G) < n_vec) val[u] = __ldg(q16 + gl + u * G);
#pragma unroll
          for (int u = 0; u < kBatch; ++u)
            if ((uint32_t)(gl + u * G) < n_vec) acc += vector_sum<ES>(val[u]);
          for (uint32_t i = gl + kBatch * G; i < n_vec; i += G) acc += vector_sum<ES>(__ldg(q16 + i));
        } else {
          for (uint32_t e = gl; e < run_len; e += G) acc += element_at<ES>(q + (size_t)e * ES);
        }
      }
    } else if (row < rows) {  // no piece holds the row whole: element by element through the functor
      amap_view_source s;
      for (uint32_t c = gl; c < cols; c += G)
        if (amap_view_locate(v, row * cols + c, &s))
          acc += s.input < 0 ? ((uint32_t)s.fill_bits & elem_mask) : element_at<ES>(ptrs.src[s.input] + s.index * ES);
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
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // rows that are whole runs of one piece each (tabulated here, on the host): the kernel that decodes once per row
  if (view->small && cols <= 0x7FFFFFFF) {
    amap_view_rows R;
    memset(&R, 0, sizeof R);
    R.usable = 1;
    R.n_pieces = view->n_pieces;
    R.cols = (uint32_t)cols;
    for (int p = 0; p < view->n_pieces && R.usable; ++p) amap_view_rows_build(*view, p, (uint32_t)cols, &R);
    if (R.usable && view->n_pieces > 0) {
      // lanes per row: a quarter of a run's 16-byte chunks (a lane takes four of them), a power of two, at most a warp
      const int64_t run_chunks = ((int64_t)R.piece[0].run_len * view->elem_size + 15) / 16;
      int G = 1;
      while (G < 32 && G * 4 < run_chunks) G <<= 1;
      const int64_t needed = (rows + kThreads / G - 1) / (kThreads / G);
      int sms = 148;
      int dev = 0;
      if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      const unsigned blocks = (unsigned)std::min<int64_t>(needed, (int64_t)sms * 16);
      switch (view->elem_size) {
        case 4: row_sums_by_runs_kernel<4><<<blocks, kThreads, 0, s>>>(*view, R, ptrs, rows, sums_dev, G); break;
        case 2: row_sums_by_runs_kernel<2><<<blocks, kThreads, 0, s>>>(*view, R, ptrs, rows, sums_dev, G); break;
        default: row_sums_by_runs_kernel<1><<<blocks, kThreads, 0, s>>>(*view, R, ptrs, rows, sums_dev, G); break;
      }
      return cudaGetLastError() == cudaSuccess ? AMAP_OK : AMAP_ECUDA;
    }
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
  switch (view->elem_size) {
    case 4: row_sums_kernel<4><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
    case 2: row_sums_kernel<2><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
    default: row_sums_kernel<1><<<(unsigned)blocks, kThreads, 0, s>>>(*view, ptrs, rows, cols, sums_dev, G, rows_per_group); break;
  }
  return cudaGetLastError() == cudaSuccess ? AMAP_OK : AMAP_ECUDA;
}

// The row tables walked on the HOST: the result written row by row from host copies of the inputs, with the very
// functions the consumer kernel uses (amap_view_rows_build, amap_view_row_seek, amap_view_row_run).  For tests.
extern "C" int amap_view_rows_gather_host(const amap_device_view *view, int64_t cols, const void *const *src_host_ptrs,
                                          void *dst_host) {
  if (!view || cols <= 0 || cols > 0x7FFFFFFF || !dst_host) return AMAP_EINVAL;
  if (view->n_pieces < 0 || view->n_pieces > AMAP_VIEW_MAX_PIECES) return AMAP_EINVAL;
  if (view->out_numel % cols) return AMAP_EINVAL;
  if (view->n_inputs > 0 && !src_host_ptrs) return AMAP_EINVAL;
  if (!view->small) return AMAP_EUNSUPPORTED;
  amap_view_rows R;
  memset(&R, 0, sizeof R);
  R.usable = 1;
  R.n_pieces = view->n_pieces;
  R.cols = (uint32_t)cols;
  for (int p = 0; p < view->n_pieces && R.usable; ++p) amap_view_rows_build(*view, p, (uint32_t)cols, &R);
  if (!R.usable) return AMAP_EUNSUPPORTED;
  const int es = view->elem_size;
  char *dst = static_cast<char *>(dst_host);
  for (int64_t row = 0; row < view->out_numel / cols; ++row) {
    amap_view_row_cursor cur;
    amap_view_row_seek(R, (uint32_t)(row * cols), &cur);
    if (cur.piece < 0) return AMAP_EUNSUPPORTED;  // a row that no piece holds whole
    const amap_view_row_piece &rp = R.piece[cur.piece];
    const uint64_t fill = ((uint64_t)rp.fill_bits_hi << 32) | rp.fill_bits_lo;
    for (int j = 0; j < rp.n_runs; ++j) {
      char *out = dst + (row * cols + (int64_t)j * rp.run_len) * es;
      uint32_t s;
      if (amap_view_row_run(rp, cur, j, &s)) {
        memcpy(out, static_cast<const char *>(src_host_ptrs[rp.input]) + (size_t)s * es, (size_t)rp.run_len * es);
      } else {
        for (int e = 0; e < rp.run_len; ++e) memcpy(out + (size_t)e * es, &fill, (size_t)es);  // little-endian host
      }
    }
  }
  return AMAP_OK;
}
