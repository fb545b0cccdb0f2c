// Low-rank sparsity predictor (Section 3.1, "Anticipating ReLU Sparsity"; Appendix B):
// scores = x.A.B + c, active iff score > theta, compacted to an ascending index list.
//
// Both stages are HBM-bound GEMVs over fp16 factors with fp32 accumulation:
//   stage 1  z_partial[p] = x[rows of p] . A[rows of p]      (A read once, 16-byte loads)
//   stage 2  score = (sum_p z_partial[p]) . B[:, tile] + c   (B read once, 16-byte loads)
// Stage 2 also thresholds (warp ballot -> bit mask) and the last CTA to finish turns the bit
// mask into the sorted list with a block prefix sum, so the list order never depends on
// scheduling.  Summation orders are fixed: results are bit-reproducible run to run.
#include "lif_internal.cuh"
#include "mask_compact.cuh"

namespace lif {
namespace {

// ---- stage 1: z_partial[cta][s][j] = sum_{m in rows(cta)} x[s][m] * A[m][j] -------------
template <int S>
__global__ void __launch_bounds__(kThreads)
predict_z_kernel(const __half* __restrict__ x, const __half* __restrict__ A, int d, int r,
                 int rows_per_cta, float* __restrict__ z_partial, int* predictor_run) {
  __shared__ float red[2048];
  const int ncg = r >> 3;            // 8-column groups (16 bytes each)
  const int nrl = kThreads / ncg;    // row lanes
  const int tid = threadIdx.x;
  const int cg = tid % ncg, rl = tid / ncg;
  const int m0 = blockIdx.x * rows_per_cta;
  const int m1 = min(d, m0 + rows_per_cta);

  float acc[S][8];
#pragma unroll
  for (int s = 0; s < S; ++s)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[s][e] = 0.f;

  // A is a weight: its first 8 rows per thread are put in flight before the dependency wait,
  // x (possibly written by the previous kernel) only after it.
  uint4 aq[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int m = m0 + rl + u * nrl;
    aq[u] = (rl < nrl && m < m1) ? ld_stream16(A + (size_t)m * r + cg * 8) : make_uint4(0, 0, 0, 0);
  }
  pdl_wait();
  pdl_trigger();
  // every earlier kernel is complete: a new predictor run begins, and its number is settled
  // before the score kernel, which tags its mask words with it, passes its own wait
  if (blockIdx.x == 0 && tid == 0) *predictor_run = (int)((unsigned)*predictor_run + 1u);   // wraps
  if (rl < nrl) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int m = m0 + rl + u * nrl;
      if (m < m1) {
        float af[8];
        unpack8(aq[u], af);
#pragma unroll
        for (int s = 0; s < S; ++s) {
          const float xs = __half2float(x[(size_t)s * d + m]);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[s][e] = fmaf(xs, af[e], acc[s][e]);
        }
      }
    }
#pragma unroll 4
    for (int m = m0 + rl + 8 * nrl; m < m1; m += nrl) {
      float af[8];
      unpack8(ld_stream16(A + (size_t)m * r + cg * 8), af);
#pragma unroll
      for (int s = 0; s < S; ++s) {
        const float xs = __half2float(x[(size_t)s * d + m]);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[s][e] = fmaf(xs, af[e], acc[s][e]);
      }
    }
  }
  // fold the row lanes, one stream at a time (8 KB of shared memory)
#pragma unroll
  for (int s = 0; s < S; ++s) {
    if (rl < nrl) {
#pragma unroll
      for (int e = 0; e < 8; ++e) red[rl * r + cg * 8 + e] = acc[s][e];
    }
    __syncthreads();
    for (int j = tid; j < r; j += kThreads) {
      float v = 0.f;
      for (int l = 0; l < nrl; ++l) v += red[l * r + j];
      z_partial[((size_t)blockIdx.x * S + s) * r + j] = v;
    }
    __syncthreads();
  }
}

// ---- stage 2: scores, threshold, bit mask; last CTA compacts ------------------------------
// kSpec: also record per neuron the last token < keep in which it is active (speculative mode).
template <int S, bool kSpec>
__global__ void __launch_bounds__(kThreads)
predict_logits_kernel(const float* __restrict__ z_partial, int P, const __half* __restrict__ B,
                      const float* __restrict__ c, float theta, int r, int F,
                      float* __restrict__ logits, uint32_t* mask_words, int* ticket,
                      int* __restrict__ active_idx, int* __restrict__ n_active, int compact,
                      int8_t* __restrict__ keep_tok, int keep, const int32_t* __restrict__ slot_of,
                      unsigned long long* new_mask_words, const int* predictor_run) {
  extern __shared__ float zs[];                 // [S][r]
  __shared__ float red[16][kLogitTile];
  __shared__ int warp_sums[kThreads / 32];
  __shared__ int is_last;
  const int tid = threadIdx.x;

  // B does not depend on stage 1: put the first 128 rows of this CTA's tile in flight before
  // touching z (8 x 16 bytes per thread), then fold the stage-1 partials while they travel.
  const int cg = tid & 15, rs = tid >> 4;
  const int col = blockIdx.x * kLogitTile + cg * 8;
  uint4 bq[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int j = rs + 16 * u;
    bq[u] = (col < F && j < r) ? ld_stream16(B + (size_t)j * F + col) : make_uint4(0, 0, 0, 0);
  }
  const int my_col = blockIdx.x * kLogitTile + tid;   // used by threads < kLogitTile
  const float my_c = (tid < kLogitTile && my_col < F) ? c[my_col] : 0.f;
  // The window state was last written by this layer's previous step, complete long before this
  // kernel could start: whether the neuron already has a cache row is read here, so the mask of
  // neurons to bring in (active and not cached) costs no round trip of its own.
  const int my_row = (tid < kLogitTile && my_col < F) ? slot_of[my_col] : 0;
  pdl_wait();
  pdl_trigger();
  const int run = (tid < kLogitTile && (tid & 31) == 0) ? __ldcg(predictor_run) : 0;
  if (S == 1) {
    // one stream: every partial of a sum is requested before the first is used (one memory
    // round trip instead of several); the additions keep their order
    for (int i = tid; i < S * r; i += kThreads) {
      float t[kMaxZPartials];
#pragma unroll
      for (int p = 0; p < kMaxZPartials; ++p)
        t[p] = p < P ? __ldcg(z_partial + (size_t)p * S * r + i) : 0.f;
      float v = 0.f;
#pragma unroll
      for (int p = 0; p < kMaxZPartials; ++p)
        if (p < P) v += t[p];
      zs[i] = v;
    }
  } else {
    // several streams: S * r sums per CTA; four per thread at a time keep 32 loads in flight
    // (same order of additions per sum)
    for (int i0 = tid; i0 < S * r; i0 += 4 * kThreads) {
      float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
      for (int p = 0; p < P; ++p) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u * kThreads;
          if (i < S * r) v[u] += __ldcg(z_partial + (size_t)p * S * r + i);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + u * kThreads < S * r) zs[i0 + u * kThreads] = v[u];
    }
  }
  __syncthreads();

  float acc[S][8];
#pragma unroll
  for (int s = 0; s < S; ++s)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[s][e] = 0.f;
  for (int j0 = 0; j0 < r; j0 += 128) {
    if (j0 > 0) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int j = j0 + rs + 16 * u;
        bq[u] = (col < F && j < r) ? ld_stream16(B + (size_t)j * F + col) : make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + rs + 16 * u;
      if (j < r) {
        float bf[8];
        unpack8(bq[u], bf);
#pragma unroll
        for (int s = 0; s < S; ++s) {
          const float zz = zs[s * r + j];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[s][e] = fmaf(zz, bf[e], acc[s][e]);
        }
      }
    }
  }

  bool active = false;
  int last_kept = -1;        // speculative mode: last token < keep in which the neuron is active
#pragma unroll
  for (int s = 0; s < S; ++s) {
#pragma unroll
    for (int e = 0; e < 8; ++e) red[rs][cg * 8 + e] = acc[s][e];
    __syncthreads();
    if (tid < kLogitTile && my_col < F) {
      float v = 0.f;
#pragma unroll
      for (int k = 0; k < 16; ++k) v += red[k][tid];
      v += my_c;
      if (logits) logits[(size_t)s * F + my_col] = v;
      active = active || (v > theta);
      if (kSpec && v > theta && s < keep) last_kept = s;
    }
    __syncthreads();
  }
  if (kSpec && tid < kLogitTile && my_col < F) keep_tok[my_col] = (int8_t)last_kept;
  if (tid < kLogitTile) {
    const unsigned m = __ballot_sync(0xffffffffu, active);
    const unsigned mn = __ballot_sync(0xffffffffu, active && my_row < 0);
    if ((tid & 31) == 0) {
      mask_words[blockIdx.x * (kLogitTile / 32) + (tid >> 5)] = m;
      // the bits together with this run's number, in one store: a fetch kernel that is already
      // resident re-reads the entry until the number is the run's
      const unsigned long long e = (unsigned long long)mn | ((unsigned long long)(unsigned)run << 32);
      asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(
                       new_mask_words + blockIdx.x * (kLogitTile / 32) + (tid >> 5)), "l"(e) : "memory");
    }
  }

  if (!compact) return;     // the consumer reads the bit mask itself
  compact_mask_last_cta(mask_words, gridDim.x * (kLogitTile / 32), ticket, active_idx, n_active,
                        warp_sums, &is_last);
}

template <int S>
cudaError_t launch_predict_s(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                             int32_t* n_active, cudaStream_t st, cudaEvent_t* ev, int compact) {
  const lif_layer_desc& D = L->desc;
  cudaError_t e = launch_k(predict_z_kernel<S>, dim3(L->z_ctas), dim3(kThreads), 0, st, L->use_pdl,
                           x, (const __half*)D.dev_pred_A, D.d_model, D.rank,
                           z_rows_per_cta(D.d_model), L->z_partial,
                           (int*)(L->counts + CNT_PREDICTOR_RUN));
  if (e != cudaSuccess) return e;
  if (ev) tm_record(ev[1], st);
  const int grid = (D.d_ff + kLogitTile - 1) / kLogitTile;
  const size_t smem = (size_t)S * D.rank * sizeof(float);
  if (smem > 32 * 1024) {
    e = cudaFuncSetAttribute(predict_logits_kernel<S, false>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(predict_logits_kernel<S, true>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  auto kernel = L->keep_tok ? predict_logits_kernel<S, true> : predict_logits_kernel<S, false>;
  e = launch_k(kernel, dim3(grid), dim3(kThreads), smem, st, L->use_pdl,
               (const float*)L->z_partial, L->z_ctas, (const __half*)D.dev_pred_B, D.dev_pred_c,
               D.threshold_logit, D.rank, D.d_ff, logits, L->mask_words,
               (int*)(L->counts + CNT_TICKET_PREDICT), (int*)active_idx, (int*)n_active, compact,
               L->keep_tok, D.spec_keep, (const int32_t*)L->slot_of, L->new_mask_words,
               (int*)(L->counts + CNT_PREDICTOR_RUN));
  if (ev) tm_record(ev[2], st);
  return e;
}

}  // namespace

cudaError_t launch_predict_one(lif_layer* L, int kernel, const __half* x, cudaStream_t st) {
  const lif_layer_desc& D = L->desc;
  if (D.n_streams != 1) return cudaErrorInvalidValue;
  if (D.gate_mode == LIF_GATE_RESIDENT)
    return kernel == LIF_KERNEL_PREDICT_SCORES
               ? launch_gate_predict(L, x, nullptr, L->active_idx, L->n_tmp, st, nullptr,
                                     L->fused_plan ? 0 : 1)
               : cudaErrorInvalidValue;
  if (kernel == LIF_KERNEL_PREDICT_Z)
    return launch_k(predict_z_kernel<1>, dim3(L->z_ctas), dim3(kThreads), 0, st, L->use_pdl, x,
                    (const __half*)D.dev_pred_A, D.d_model, D.rank, z_rows_per_cta(D.d_model),
                    L->z_partial, (int*)(L->counts + CNT_PREDICTOR_RUN));
  const int grid = (D.d_ff + kLogitTile - 1) / kLogitTile;
  return launch_k(L->keep_tok ? predict_logits_kernel<1, true> : predict_logits_kernel<1, false>,
                  dim3(grid), dim3(kThreads),
                  (size_t)D.rank * sizeof(float), st, L->use_pdl, (const float*)L->z_partial,
                  L->z_ctas, (const __half*)D.dev_pred_B, D.dev_pred_c, D.threshold_logit, D.rank,
                  D.d_ff, (float*)nullptr, L->mask_words, (int*)(L->counts + CNT_TICKET_PREDICT),
                  (int*)L->active_idx, (int*)L->n_tmp, L->fused_plan ? 0 : 1, L->keep_tok,
                  D.spec_keep, (const int32_t*)L->slot_of, L->new_mask_words,
                  (int*)(L->counts + CNT_PREDICTOR_RUN));
}

cudaError_t launch_predict(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                           int32_t* n_active, cudaStream_t st, cudaEvent_t* ev, int compact) {
  if (L->desc.gate_mode == LIF_GATE_RESIDENT)
    return launch_gate_predict(L, x, logits, active_idx, n_active, st, ev, compact);
  switch (L->desc.n_streams) {
    case 1: return launch_predict_s<1>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 2: return launch_predict_s<2>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 3: return launch_predict_s<3>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 4: return launch_predict_s<4>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 5: return launch_predict_s<5>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 6: return launch_predict_s<6>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 7: return launch_predict_s<7>(L, x, logits, active_idx, n_active, st, ev, compact);
    case 8: return launch_predict_s<8>(L, x, logits, active_idx, n_active, st, ev, compact);
  }
  return cudaErrorInvalidValue;
}

}  // namespace lif
