// The resident gate projection as the predictor (Appendix C, Llama 2, "alternative
// approaches"): with a gated FFN whose activation makes the gate values sparse, the gate
// projection kept in device memory gives the exact gate pre-activation of every neuron,
//   g[s][i] = <gate_i, x[s]> + bias_i,
// a neuron is active iff g exceeds the activation's threshold for at least one stream, and the
// FFN reuses g instead of recomputing it.  A dense fp16 GEMV over [d_ff][d_model] with fp32
// accumulation: every gate row is read once with 16-byte loads.  A CTA owns 32 consecutive
// neurons (one word of the bit mask; 8 or 16, whole bytes of it, are possible too), a warp four
// of them, so a thread keeps four independent rows in flight.  Bound: HBM bandwidth,
// 2*d_model bytes per neuron.
#include "lif_internal.cuh"
#include "mask_compact.cuh"

namespace lif {
namespace {

#ifndef LIF_GATE_ROWS
#define LIF_GATE_ROWS 4
#endif
#ifndef LIF_GATE_DEPTH
#define LIF_GATE_DEPTH 2
#endif
constexpr int kRowsPerWarp = LIF_GATE_ROWS;           // 1, 2 or 4
constexpr int kGateTile = 8 * kRowsPerWarp;           // neurons per CTA: 1, 2 or 4 bytes of the mask
constexpr int kDepth = LIF_GATE_DEPTH;   // load groups in flight per lane (one 16-byte piece per row each)

template <int S>
__global__ void __launch_bounds__(kThreads)
gate_scores_kernel(const __half* __restrict__ x, const __half* __restrict__ gate,
                   const __half* __restrict__ bias, float theta, int d, int F,
                   float* __restrict__ gate_val, float* __restrict__ logits,
                   uint32_t* mask_words, int* ticket, int* __restrict__ active_idx,
                   int* __restrict__ n_active, int compact, int nwords,
                   const int32_t* __restrict__ slot_of, unsigned long long* new_mask_words,
                   const int* predictor_run) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);          // [S][d / 8]
  __shared__ int act_flag[kGateTile];     // bit 0: active, bit 1: active and not cached yet
  __shared__ int warp_sums[kThreads / 32];
  __shared__ int is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = d >> 3;
  const int i0 = blockIdx.x * kGateTile + warp * kRowsPerWarp;   // this warp's first neuron

  // Each lane keeps kDepth groups of loads in flight, a group being one 16-byte piece of each of
  // its rows.  The gate rows are weights: the first groups are issued before the
  // dependency wait; x (possibly written by the previous kernel) comes after it.
  const int ngroups = (nvec + 31) >> 5;
  auto load_group = [&](uint4* dst, int g) {
    const int c = lane + 32 * g;
#pragma unroll
    for (int q = 0; q < kRowsPerWarp; ++q)
      dst[q] = (i0 + q < F && c < nvec) ? ld_stream16(gate + (size_t)(i0 + q) * d + c * 8)
                                        : make_uint4(0, 0, 0, 0);
  };
  uint4 w[kDepth][kRowsPerWarp];
#pragma unroll
  for (int j = 0; j < kDepth; ++j) load_group(w[j], j);
  pdl_wait();
  pdl_trigger();
  const int run = tid == 0 ? __ldcg(predictor_run) : 0;
  for (int c = tid; c < S * nvec; c += kThreads) xs[c] = reinterpret_cast<const uint4*>(x)[c];
  __syncthreads();

  float acc[kRowsPerWarp][S];
#pragma unroll
  for (int q = 0; q < kRowsPerWarp; ++q)
#pragma unroll
    for (int s = 0; s < S; ++s) acc[q][s] = 0.f;

  for (int g0 = 0; g0 < ngroups; g0 += kDepth) {
#pragma unroll
    for (int j = 0; j < kDepth; ++j) {
      const int c = lane + 32 * (g0 + j);
      if (c < nvec) {
        float wf[kRowsPerWarp][8];
#pragma unroll
        for (int q = 0; q < kRowsPerWarp; ++q) unpack8(w[j][q], wf[q]);
#pragma unroll
        for (int s = 0; s < S; ++s) {
          float xf[8];
          unpack8(xs[s * nvec + c], xf);
#pragma unroll
          for (int q = 0; q < kRowsPerWarp; ++q)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[q][s] = fmaf(wf[q][e], xf[e], acc[q][s]);
        }
      }
      load_group(w[j], g0 + j + kDepth);     // past the end of the row: no load, zeros
    }
  }

  // warp sums in a fixed order; lane q finishes neuron i0 + q
#pragma unroll
  for (int q = 0; q < kRowsPerWarp; ++q)
#pragma unroll
    for (int s = 0; s < S; ++s) {
      float v = acc[q][s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      acc[q][s] = v;
    }
  if (lane < kRowsPerWarp) {
    const int i = i0 + lane;
    bool active = false;
    if (i < F) {
      const float b = __half2float(bias[i]);
#pragma unroll
      for (int s = 0; s < S; ++s) {
        float v = 0.f;
#pragma unroll
        for (int q = 0; q < kRowsPerWarp; ++q)
          if (q == lane) v = acc[q][s];
        v += b;
        gate_val[(size_t)s * F + i] = v;
        if (logits) logits[(size_t)s * F + i] = v;
        active = active || (v > theta);
      }
    }
    // (the window state of the previous step is final long before this kernel starts)
    act_flag[warp * kRowsPerWarp + lane] = active ? (slot_of[i] < 0 ? 3 : 1) : 0;
  }
  __syncthreads();
  if (warp == 0) {
    // the CTA's 8, 16 or 32 bits are whole bytes of the mask: a plain store, no merging
    const unsigned m = __ballot_sync(0xffffffffu, lane < kGateTile && act_flag[lane] != 0);
    const unsigned mn = __ballot_sync(0xffffffffu, lane < kGateTile && (act_flag[lane] & 2));
    if (lane == 0) {
      if (kGateTile == 32) {
        mask_words[blockIdx.x] = m;
      } else if (kGateTile == 16) {
        reinterpret_cast<uint16_t*>(mask_words)[blockIdx.x] = (uint16_t)m;
      } else {
        reinterpret_cast<uint8_t*>(mask_words)[blockIdx.x] = (uint8_t)m;
      }
      // this CTA's neurons to bring in, with the run's number, in one store (one entry per CTA):
      // a fetch kernel that is already resident re-reads the entry until the number is the run's
      const unsigned long long e = (unsigned long long)mn | ((unsigned long long)(unsigned)run << 32);
      asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(new_mask_words + blockIdx.x), "l"(e)
                   : "memory");
    }
  }
  if (!compact) return;     // the consumer reads the bit mask itself
  compact_mask_last_cta(mask_words, nwords, ticket, active_idx, n_active, warp_sums, &is_last);
}

template <int S>
cudaError_t launch_gate_s(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                          int32_t* n_active, cudaStream_t st, int compact) {
  const lif_layer_desc& D = L->desc;
  const int grid = (D.d_ff + kGateTile - 1) / kGateTile;
  const size_t smem = (size_t)S * D.d_model * 2;
  if (smem > 32 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(gate_scores_kernel<S>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const float theta = D.activation == LIF_ACT_FATRELU ? D.activation_threshold : 0.f;
  return launch_k(gate_scores_kernel<S>, dim3(grid), dim3(kThreads), smem, st, L->use_pdl, x,
                  (const __half*)D.dev_gate, (const __half*)D.dev_bias_up, theta, D.d_model,
                  D.d_ff, L->gate_val, logits, L->mask_words,
                  (int*)(L->counts + CNT_TICKET_PREDICT), (int*)active_idx, (int*)n_active, compact,
                  (D.d_ff + 31) / 32, (const int32_t*)L->slot_of, L->new_mask_words,
                  (int*)(L->counts + CNT_PREDICTOR_RUN));
}

}  // namespace

int gate_predict_tile() { return kGateTile; }

cudaError_t launch_gate_predict(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                                int32_t* n_active, cudaStream_t st, cudaEvent_t* ev, int compact) {
  if (ev) tm_record(ev[1], st);     // no first stage in this mode
  cudaError_t e = cudaErrorInvalidValue;
  switch (L->desc.n_streams) {
    case 1: e = launch_gate_s<1>(L, x, logits, active_idx, n_active, st, compact); break;
    case 2: e = launch_gate_s<2>(L, x, logits, active_idx, n_active, st, compact); break;
    case 3: e = launch_gate_s<3>(L, x, logits, active_idx, n_active, st, compact); break;
    case 4: e = launch_gate_s<4>(L, x, logits, active_idx, n_active, st, compact); break;
    case 5: e = launch_gate_s<5>(L, x, logits, active_idx, n_active, st, compact); break;
    case 6: e = launch_gate_s<6>(L, x, logits, active_idx, n_active, st, compact); break;
    case 7: e = launch_gate_s<7>(L, x, logits, active_idx, n_active, st, compact); break;
    case 8: e = launch_gate_s<8>(L, x, logits, active_idx, n_active, st, compact); break;
  }
  if (ev) tm_record(ev[2], st);
  return e;
}

}  // namespace lif
