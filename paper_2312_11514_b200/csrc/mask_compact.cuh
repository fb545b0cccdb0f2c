// Bit mask -> ascending index list, done by the last CTA of a grid to finish (shared by the
// low-rank predictor and the resident-gate predictor).
#pragma once

#include "lif_internal.cuh"

namespace lif {

__device__ __forceinline__ int block_exclusive_scan_256(int v, int* total, int* warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    int ws = warp_sums[w];
    if (w < warp) base += ws;
    tot += ws;
  }
  *total = tot;
  __syncthreads();
  return base + inc - v;
}

// Every CTA calls this after writing its words of `mask_words`.  The CTA that draws the last
// ticket prefix-sums the whole mask (nwords words) into active_idx / n_active and re-arms the
// ticket; the list order never depends on scheduling.  warp_sums: kThreads / 32 ints and
// is_last: one int, both in shared memory.
__device__ __forceinline__ void compact_mask_last_cta(const uint32_t* mask_words, int nwords,
                                                      int* ticket, int* __restrict__ active_idx,
                                                      int* __restrict__ n_active, int* warp_sums,
                                                      int* is_last) {
  const int tid = threadIdx.x;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int t = atomicAdd(ticket, 1);
    *is_last = (t == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (!*is_last) return;
  __threadfence();

  const int wpt = (nwords + kThreads - 1) / kThreads;
  const int w0 = min(nwords, tid * wpt), w1 = min(nwords, w0 + wpt);
  int cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(__ldcg(mask_words + w));
  int total;
  int off = block_exclusive_scan_256(cnt, &total, warp_sums);
  for (int w = w0; w < w1; ++w) {
    unsigned m = __ldcg(mask_words + w);
    while (m) {
      const int b = __ffs(m) - 1;
      active_idx[off++] = w * 32 + b;
      m &= m - 1;
    }
  }
  if (tid == 0) {
    *n_active = total;
    *ticket = 0;
  }
}

}  // namespace lif
