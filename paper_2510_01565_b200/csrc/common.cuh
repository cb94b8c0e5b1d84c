// Types shared by the kernels of libdit.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dit.h"

namespace dit {

// Packed-batch description, passed by value as a kernel parameter (no device-side plan buffer):
// cu[r] .. cu[r+1] are the packed rows of request r.  `order` lists requests longest first (used by
// the attention grid so that long requests start early).
struct SeqInfo {
  int n;
  int total;
  int cu[DIT_MAX_REQUESTS + 1];
  int order[DIT_MAX_REQUESTS];
};

// Image geometry of the packed requests, for kernels that need a token's patch row and column:
// the first img_cu[r+1] - img_cu[r] rows of request r are its image tokens in row-major patch order,
// gw[r] patches per row; the rest are text tokens (position (0, 0)).
struct RowGeom {
  int img_cu[DIT_MAX_REQUESTS + 1];
  int gw[DIT_MAX_REQUESTS];
};

// Device status word values (written by a kernel whose bounded wait ran out).
enum : int { kStatusOk = 0, kStatusGemmTimeout = 1, kStatusAttnTimeout = 2, kStatusLnTimeout = 3, kStatusModTimeout = 4, kStatusTestTimeout = 5 };

// Request that owns packed row `row` (binary search over at most 64 entries).
__device__ __forceinline__ int find_request(const SeqInfo& s, int row) {
  int lo = 0, hi = s.n - 1;
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (s.cu[mid] <= row) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// 0 for an image token, 1 for a text token (two-stream blocks choose their tensors by this).
__device__ __forceinline__ int row_kind(const SeqInfo& s, const RowGeom& g, int req, int row) {
  return (row - s.cu[req]) >= (g.img_cu[req + 1] - g.img_cu[req]) ? 1 : 0;
}

}  // namespace dit
