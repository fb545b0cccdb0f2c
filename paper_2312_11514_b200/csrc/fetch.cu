// Bringing in new neurons (Section 3.3 item 2): gather the bundles of the newly needed
// neurons from the full store in mapped pinned host memory (standing in for flash) into
// their cache rows.  The kernel reads host memory directly: every warp instruction reads 512
// contiguous bytes of one bundle with 16-byte loads, and each thread keeps several loads in
// flight so the link sees enough outstanding requests.  Bound: host-link bandwidth.
#include "lif_internal.cuh"

namespace lif {
namespace {

constexpr int kFetchUnroll = 8;   // 16-byte loads in flight per thread

__device__ __forceinline__ uint4 ld_host(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Copies `row_vec` 16-byte vectors per row.  Work unit = (row, slice of kThreads*kFetchUnroll
// vectors); units are dealt round-robin to CTAs so a short list still spreads over the grid.
__device__ __forceinline__ void gather_rows(const uint4* __restrict__ src_base,
                                            uint4* __restrict__ dst_base,
                                            const int32_t* __restrict__ src_rows,
                                            const int32_t* __restrict__ dst_rows, int n,
                                            int row_vec) {
  constexpr int kSlice = kThreads * kFetchUnroll;
  const int slices = (row_vec + kSlice - 1) / kSlice;
  const long long units = (long long)n * slices;
  for (long long u = blockIdx.x; u < units; u += gridDim.x) {
    const int j = (int)(u / slices);
    const int v0 = (int)(u % slices) * kSlice + threadIdx.x;
    const long long srow = src_rows ? src_rows[j] : j;
    const long long drow = dst_rows ? dst_rows[j] : j;
    const uint4* src = src_base + srow * row_vec;
    uint4* dst = dst_base + drow * row_vec;
    uint4 buf[kFetchUnroll];
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = v0 + i * kThreads;
      if (v < row_vec) buf[i] = ld_host(src + v);
    }
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = v0 + i * kThreads;
      if (v < row_vec) dst[v] = buf[i];
    }
  }
}

__global__ void __launch_bounds__(kThreads)
fetch_kernel(const uint4* __restrict__ store, uint4* __restrict__ cache,
             const int32_t* __restrict__ load_ids, const int32_t* __restrict__ load_slots,
             const int32_t* __restrict__ counts, int row_vec) {
  pdl_wait();
  pdl_trigger();
  gather_rows(store, cache, load_ids, load_slots, counts[LIF_CNT_N_LOAD], row_vec);
}

__global__ void __launch_bounds__(kThreads)
probe_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n_chunks,
             int chunk_vec) {
  gather_rows(src, dst, nullptr, nullptr, n_chunks, chunk_vec);
}

// Refill after a restore: cache row s <- bundle pointers[s] for s < num_used.
__global__ void __launch_bounds__(kThreads)
refill_kernel(const uint4* __restrict__ store, uint4* __restrict__ cache,
              const int32_t* __restrict__ pointers, const int32_t* __restrict__ counts,
              int row_vec) {
  gather_rows(store, cache, pointers, nullptr, counts[LIF_CNT_NUM_USED], row_vec);
}

}  // namespace

cudaError_t launch_refill(lif_layer* L, cudaStream_t st) {
  refill_kernel<<<L->fetch_grid, kThreads, 0, st>>>((const uint4*)L->dev_bundles,
                                                    (uint4*)L->desc.dev_cache, L->pointers,
                                                    L->counts, row_elems(L->desc) / 8);
  return cudaGetLastError();
}

cudaError_t launch_fetch(lif_layer* L, cudaStream_t st) {
  return launch_k(fetch_kernel, dim3(L->fetch_grid), dim3(kThreads), 0, st, L->use_pdl,
                  (const uint4*)L->dev_bundles, (uint4*)L->desc.dev_cache,
                  (const int32_t*)L->load_ids, (const int32_t*)L->load_slots,
                  (const int32_t*)L->counts, row_elems(L->desc) / 8);
}

cudaError_t launch_probe(const void* dev_src_alias, void* dev_dst, size_t bytes, size_t chunk,
                         int grid, cudaStream_t st) {
  probe_kernel<<<grid, kThreads, 0, st>>>((const uint4*)dev_src_alias, (uint4*)dev_dst,
                                          (int)(bytes / chunk), (int)(chunk / 16));
  return cudaGetLastError();
}

}  // namespace lif
