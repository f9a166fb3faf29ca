// Block-wide building blocks of the per-expert capacity select (stages 2 and 3): an exclusive
// prefix sum over a 1024-thread block and the search for the histogram bin that holds the
// rank-th largest key.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace capmoe {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int RADIX_BINS = 2048;                     // 11 + 11 + 10 bits

// Exclusive prefix sum over the block (SEL_THREADS threads).  total = sum of all v.
__device__ __forceinline__ uint32_t block_scan(uint32_t v, uint32_t* sh /*[SEL_WARPS+1]*/, uint32_t& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) sh[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    uint32_t w = sh[lane];                       // SEL_WARPS == 32
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    sh[lane] = wi - w;
    if (lane == 31) sh[SEL_WARPS] = wi;
  }
  __syncthreads();
  const uint32_t res = incl - v + sh[wid];
  total = sh[SEL_WARPS];
  __syncthreads();                               // sh may be reused right away
  return res;
}

// Among `nbins` histogram bins ordered from the highest digit down, find the bin that holds the
// rank-th largest element (rank >= 1).  Result in out[0] = bin, out[1] = rank inside that bin.
__device__ __forceinline__ void find_bin(const int* hist, int nbins, uint32_t rank, uint32_t* scan_sh,
                                         uint32_t* out) {
  const int p0 = 2 * threadIdx.x, p1 = p0 + 1;
  const uint32_t h0 = p0 < nbins ? (uint32_t)hist[nbins - 1 - p0] : 0u;
  const uint32_t h1 = p1 < nbins ? (uint32_t)hist[nbins - 1 - p1] : 0u;
  uint32_t total;
  const uint32_t before = block_scan(h0 + h1, scan_sh, total);
  if (before < rank && rank <= before + h0) {
    out[0] = (uint32_t)(nbins - 1 - p0); out[1] = rank - before;
  } else if (before + h0 < rank && rank <= before + h0 + h1) {
    out[0] = (uint32_t)(nbins - 1 - p1); out[1] = rank - before - h0;
  }
  __syncthreads();
}

}  // namespace capmoe
