// The exchange of a neuron-sharded layer-step.  With a layer's neurons split over several
// devices each device holds the sum of the FFN terms of its own neurons (Section 3.3 item 3:
// the output is one term per cached neuron, in any order), and the layer's output is the sum
// of those partial outputs.  This kernel forms it on the calling device by reading every
// device's partial with plain 16-byte loads -- its own from local memory, the others through
// peer mappings -- and adding them in rank order, so every device gets the same bits.  No
// multicast or bulk-tensor load is involved: peers are read with ld.global only.
// Bound: launch latency (n_peers x [S][d] fp32, 16 KiB each at d_model 4096).
#include "lif_internal.cuh"

namespace lif {
namespace {

struct PeerPartials {
  const float4* p[LIF_MAX_PEERS];
};

__global__ void __launch_bounds__(kThreads)
sum_peer_outputs_kernel(PeerPartials src, int n_peers, float4* y, size_t n_vec) {
  pdl_wait();
  pdl_trigger();
  for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n_vec;
       i += (size_t)gridDim.x * kThreads) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // fully unrolled so that the pointers stay in the parameter bank (no local copy)
#pragma unroll
    for (int g = 0; g < LIF_MAX_PEERS; ++g) {
      if (g < n_peers) {
        // .cg: a peer's partial was written by another device; never serve it from this SM's L1
        const float4 v = __ldcg(src.p[g] + i);
        acc.x += v.x;
        acc.y += v.y;
        acc.z += v.z;
        acc.w += v.w;
      }
    }
    y[i] = acc;
  }
}

}  // namespace
}  // namespace lif

extern "C" lif_status lif_sum_peer_outputs(const float* const* dev_partials, int32_t n_peers,
                                           float* dev_y, size_t n_floats, void* stream) {
  using namespace lif;
  if (!dev_partials || !dev_y || n_peers < 1 || n_peers > LIF_MAX_PEERS || n_floats == 0 ||
      n_floats % 4)
    return LIF_ERR_INVALID_ARG;
  PeerPartials src = {};
  for (int g = 0; g < n_peers; ++g) {
    if (!dev_partials[g]) return LIF_ERR_INVALID_ARG;
    if ((uintptr_t)dev_partials[g] % 16) return LIF_ERR_ALIGNMENT;
    src.p[g] = reinterpret_cast<const float4*>(dev_partials[g]);
  }
  if ((uintptr_t)dev_y % 16) return LIF_ERR_ALIGNMENT;
  const size_t n_vec = n_floats / 4;
  size_t grid = (n_vec + kThreads - 1) / kThreads;
  if (grid > 1184) grid = 1184;   // 8 CTAs per SM on a 148-SM part; the loop strides beyond
  cudaError_t e = launch_k(sum_peer_outputs_kernel, dim3((unsigned)grid), dim3(kThreads), 0,
                           (cudaStream_t)stream, 0, src, (int)n_peers,
                           reinterpret_cast<float4*>(dev_y), n_vec);
  return e == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}
