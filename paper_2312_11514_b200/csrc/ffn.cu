// Sparse FFN over cached row-column bundles (Section 3.3 item 3):
//   y = b_down + sum_q relu(<M[slot_q, :d], x> + bias[slot_q]) * M[slot_q, d:]
// Gated layers (Appendix C, Llama 2): rows are gate | up | down and the row's weight is
// act(<gate, x> + bias) * <up, x>; or, with the gate projection resident, rows are up | down and
// the gate value of the row's neuron comes from the predictor's score array.
// A bundle is one contiguous 4*d_model-byte row (Section 3.2), so the unit of HBM traffic is
// one bulk asynchronous copy (TMA, cp.async.bulk) of a whole row into shared memory.  Each
// CTA owns rows q = cta, cta + G, ...; it issues the copies for all its rows up front (up to
// `stages` in flight); each of the 8 warps takes a row of the round and, when that row's
// mbarrier completes, dots the whole up half with x (16-byte shared loads, warp-shuffle sum)
// and applies bias + ReLU; then all 256 threads axpy the down halves into fp32 register
// accumulators.  Rows whose ReLU is zero skip the axpy.
// CTA partials go to a [G][d] fp32 scratch; a second kernel adds them in CTA order, so the
// result does not depend on scheduling.  Bound: HBM bandwidth, 4*d_model bytes per row.
#include <mutex>

#include "lif_internal.cuh"

namespace lif {
namespace {

constexpr int kMaxChunks = 4;            // 8-column chunks per thread: d_model <= 8192

struct FfnArgs {
  const __half* cache;
  const __half* bias;
  const __half* x;
  const int32_t* slots;   // or nullptr: rows base .. base + n
  const int32_t* n;
  const int32_t* base;    // or nullptr: 0
  float* y_partial;       // [gridDim.x][d]
  int32_t* status;
  int d;
  int stages;
  int slots_len;          // entries of `slots` that may be read before n is known (0: none)
  int act;                // LIF_ACT_*
  float act_thr;
  const float* gate_val;  // resident gate: this stream's gate pre-activations, by neuron id
  const int32_t* pointers;  // resident gate: row -> neuron id
  int rows;               // rows of `cache`: a slot outside [0, rows) is refused, not read
  unsigned wait_polls;    // poll limit of the first wait on each copy (kWaitLimit)
};

// kGate = LIF_GATE_*: none (row = up | down), bundled (gate | up | down), resident (up | down,
// gate value looked up by neuron id).
// (registers capped at 128 per thread, not for a second CTA of this kernel — shared memory allows
// one — but so that a CTA of it fits on an SM beside a CTA of the fetch kernel, which holds
// every SM for the length of the host-link transfer)
template <int kGate>
__global__ void __launch_bounds__(kThreads, 2) sparse_ffn_kernel(FfnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = a.d;
  constexpr int kVec = kGate == LIF_GATE_BUNDLED ? 3 : 2;       // d-vectors per row
  const unsigned row_bytes = 2u * kVec * d;
  const int stages = a.stages;
  // shared layout: rows[stages][row_bytes] | x[d] fp16 | bars[stages] | row flags[stages] |
  //                h[stages] | bias[stages]
  unsigned char* rows = smem;
  __half* xs = reinterpret_cast<__half*>(rows + (size_t)stages * row_bytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(xs) +
                                               (((size_t)d * 2 + 15) & ~(size_t)15));
  int* ok_s = reinterpret_cast<int*>(bars + stages);      // 0: the row's index was refused
  float* hs = reinterpret_cast<float*>(ok_s + stages);
  float* bias_s = hs + stages;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int nvec = d >> 3;                    // 16-byte chunks per half row

  // nothing below the wait may depend on earlier kernels of the stream
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();

  // One memory round trip for the row count and this CTA's first slots: thread i reads the
  // slot of its row before n is known when the list is long enough to make that safe.
  int my_slot = -1;
  if (tid < stages && a.slots) {
    const int q = cta + tid * G;
    if (q < a.slots_len) my_slot = a.slots[q];
  }
  // Row count and rows come from the caller (or from lists the caller could have overwritten):
  // a count outside [0, rows] is clamped and a row outside [0, rows) contributes nothing and is
  // never read; either sets LIF_ERR_INVALID_ARG in the status word.
  int n = *a.n;
  int bad_input = 0;
  if (n < 0 || n > a.rows) {
    bad_input = 1;
    n = n < 0 ? 0 : a.rows;
  }
  if (cta >= n) {                             // the reduction only reads min(G, n) partials
    if (bad_input && cta == 0 && tid == 0) atomicCAS(a.status, LIF_OK, LIF_ERR_INVALID_ARG);
    return;
  }
  const int base = a.base ? *a.base : 0;
  const int my_cnt = (n - cta + G - 1) / G;
  __syncthreads();                            // barrier init visible

  float acc[kMaxChunks][8];
#pragma unroll
  for (int c = 0; c < kMaxChunks; ++c)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[c][e] = 0.f;

  unsigned parity = 0;
  int timed_out = 0;
  for (int r0 = 0; r0 < my_cnt; r0 += stages) {
    const int rc = min(stages, my_cnt - r0);
    // thread i issues the copy of row i of this round and fetches its bias
    bool row_ok = true;
    if (tid < rc) {
      const int q = cta + (r0 + tid) * G;
      int slot;
      if (!a.slots) slot = base + q;
      else if (r0 == 0 && q < a.slots_len) slot = my_slot;
      else slot = a.slots[q];
      if (slot < 0 || slot >= a.rows) {       // refused: row 0 travels in its place, weight 0
        row_ok = false;
        bad_input = 1;
        slot = 0;
      }
      mbar_expect_tx(bars + tid, row_bytes);
      bulk_g2s(rows + (size_t)tid * row_bytes, a.cache + (size_t)slot * kVec * d, row_bytes,
               bars + tid);
      bias_s[tid] = kGate == LIF_GATE_RESIDENT ? a.gate_val[a.pointers[slot]]
                                               : __half2float(a.bias[slot]);
      ok_s[tid] = row_ok ? 1 : 0;
    }
    if (r0 == 0) {
      const uint4* xg = reinterpret_cast<const uint4*>(a.x);
      for (int c = tid; c < nvec; c += kThreads) reinterpret_cast<uint4*>(xs)[c] = xg[c];
    }
    __syncthreads();                          // x, biases and row flags of this round
    // up projection: warp w takes rows w, w + 8, ... of the round, each as soon as it has landed
    // (a whole dot product per warp: no partial sums to exchange, and the rows of a round are
    // worked on side by side instead of one after the other)
    for (int i = warp; i < rc; i += kThreads / 32) {
      if (!mbar_wait(bars + i, parity, a.wait_polls)) timed_out = 1;
      const uint4* up = reinterpret_cast<const uint4*>(rows + (size_t)i * row_bytes);
      float p = 0.f, p2 = 0.f;
#pragma unroll 4
      for (int c = lane; c < nvec; c += 32) {
        float uf[8], xf[8];
        unpack8(up[c], uf);
        unpack8(reinterpret_cast<const uint4*>(xs)[c], xf);
#pragma unroll
        for (int e = 0; e < 8; ++e) p = fmaf(uf[e], xf[e], p);
        if (kGate == LIF_GATE_BUNDLED) {       // first vector = gate row, second = up row
          unpack8(up[nvec + c], uf);
#pragma unroll
          for (int e = 0; e < 8; ++e) p2 = fmaf(uf[e], xf[e], p2);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
      if (kGate == LIF_GATE_BUNDLED) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) p2 += __shfl_xor_sync(0xffffffffu, p2, o);
      }
      if (lane == 0) {
        float h;
        if (kGate == LIF_GATE_NONE) h = apply_activation(p + bias_s[i], a.act, a.act_thr);
        else if (kGate == LIF_GATE_BUNDLED) h = apply_activation(p + bias_s[i], a.act, a.act_thr) * p2;
        else h = apply_activation(bias_s[i], a.act, a.act_thr) * p;
        hs[i] = ok_s[i] ? h : 0.f;            // a refused row contributes nothing
      }
    }
    if (__syncthreads_or(timed_out)) {        // also publishes hs[]
      // A copy did not arrive in time: flag it, give the copies still in flight one more
      // bounded chance to land (they target this CTA's shared memory), and leave.  The
      // partial is not written.
      if (tid == 0) {
        atomicCAS(a.status, LIF_OK, LIF_ERR_TIMEOUT);
        for (int i = 0; i < rc; ++i) mbar_wait(bars + i, parity);
      }
      __syncthreads();
      return;
    }
    // down projection: y += h * down half
    for (int i = 0; i < rc; ++i) {
      const float h = hs[i];
      if (h == 0.f) continue;
      const uint4* down =
          reinterpret_cast<const uint4*>(rows + (size_t)i * row_bytes) + (kVec - 1) * nvec;
#pragma unroll
      for (int k = 0; k < kMaxChunks; ++k) {
        const int c = tid + k * kThreads;
        if (c < nvec) {
          float df[8];
          unpack8(down[c], df);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[k][e] = fmaf(h, df[e], acc[k][e]);
        }
      }
    }
    __syncthreads();          // rows are free for the next round's copies
    parity ^= 1u;
  }

  if (bad_input) atomicCAS(a.status, LIF_OK, LIF_ERR_INVALID_ARG);
  float4* out = reinterpret_cast<float4*>(a.y_partial + (size_t)cta * d);
#pragma unroll
  for (int k = 0; k < kMaxChunks; ++k) {
    const int c = tid + k * kThreads;
    if (c < nvec) {
      out[2 * c] = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
      out[2 * c + 1] = make_float4(acc[k][4], acc[k][5], acc[k][6], acc[k][7]);
    }
  }
}

// y[m] = (accumulate ? y[m] : b_down[m]) + sum over set 0 then set 1 of the CTA partials
// (set j holds min(G, *n_j) partials; set 1 is optional).  A CTA owns 8 float4 columns (one
// 128-byte line per partial) x 32 slices of the partial index; each slice adds its partials
// in ascending order, then the slices are added in ascending order: a fixed summation order.
constexpr int kSumThreads = 256;
constexpr int kSumCols = 8;                     // float4 columns per CTA
__global__ void __launch_bounds__(kSumThreads)
ffn_reduce_kernel(const float* __restrict__ p0, const int32_t* __restrict__ n0,
                  const float* __restrict__ p1, const int32_t* __restrict__ n1, int G,
                  const __half* __restrict__ b_down, int b_period, float* __restrict__ y, int d,
                  int accumulate, int n_cap, int* next_run_after_wait) {
  __shared__ float4 red[32][kSumCols];
  const int tid = threadIdx.x;
  const int c4 = tid & (kSumCols - 1), gs = tid / kSumCols;
  const int col4 = blockIdx.x * kSumCols + c4;  // float4 column
  const bool in = col4 * 4 < d;
  float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
  if (gs == 0 && in) {                          // independent of earlier kernels' partials
    if (b_down && !accumulate) {
      const __half2* b = reinterpret_cast<const __half2*>(b_down + (col4 * 4) % b_period);
      const float2 lo = __half22float2(b[0]), hi = __half22float2(b[1]);
      t = make_float4(lo.x, lo.y, hi.x, hi.y);
    }
  }
  pdl_wait();
  pdl_trigger();
  // every earlier kernel of the step is complete: the next predictor run gets its number here,
  // long before it starts (a predictor without a first stage of its own relies on this)
  if (next_run_after_wait && blockIdx.x == 0 && tid == 0)
    *next_run_after_wait = (int)((unsigned)*next_run_after_wait + 1u);   // wraps
  // counts as the kernels that wrote the partials clamp them: [0, n_cap]
  const int v0 = min(G, max(0, min(*n0, n_cap))), v1 = p1 ? min(G, max(0, min(*n1, n_cap))) : 0;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (in) {
    // batches of 10 partials per thread (two sets of up to 148 over 32 slices), a batch's loads
    // in flight together; the additions keep their order
    for (int g0 = gs; g0 < v0 + v1; g0 += 32 * 10) {
      float4 v[10];
#pragma unroll
      for (int k = 0; k < 10; ++k) {
        const int g = g0 + 32 * k;
        if (g < v0 + v1) {
          const float* src = g < v0 ? p0 + (size_t)g * d : p1 + (size_t)(g - v0) * d;
          v[k] = __ldcg(reinterpret_cast<const float4*>(src) + col4);
        }
      }
#pragma unroll
      for (int k = 0; k < 10; ++k) {
        if (g0 + 32 * k < v0 + v1) {
          s.x += v[k].x; s.y += v[k].y; s.z += v[k].z; s.w += v[k].w;
        }
      }
    }
  }
  red[gs][c4] = s;
  __syncthreads();
  if (gs == 0 && in) {
    if (accumulate) t = reinterpret_cast<float4*>(y)[col4];
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      t.x += red[k][c4].x; t.y += red[k][c4].y; t.z += red[k][c4].z; t.w += red[k][c4].w;
    }
    reinterpret_cast<float4*>(y)[col4] = t;
  }
}

size_t ffn_smem_bytes(int d, int stages, int gate_mode = LIF_GATE_NONE) {
  const bool bundled = gate_mode == LIF_GATE_BUNDLED;
  size_t b = (size_t)stages * (bundled ? 6 : 4) * d;   // rows
  b += ((size_t)d * 2 + 15) & ~(size_t)15;        // x
  b += (size_t)stages * 8;                        // barriers
  b += (size_t)stages * (bundled ? 16 : 8) * 4 + (size_t)stages * 4 + (size_t)stages * 4;
  return b + 16;
}

using FfnKernel = void (*)(FfnArgs);
FfnKernel ffn_kernel_for(int gate_mode) {
  if (gate_mode == LIF_GATE_BUNDLED) return sparse_ffn_kernel<LIF_GATE_BUNDLED>;
  if (gate_mode == LIF_GATE_RESIDENT) return sparse_ffn_kernel<LIF_GATE_RESIDENT>;
  return sparse_ffn_kernel<LIF_GATE_NONE>;
}

}  // namespace

size_t ffn_smem_for(const lif_layer* L, int stages) {
  return ffn_smem_bytes(L->desc.d_model, stages, L->desc.gate_mode);
}

cudaError_t ffn_configure(lif_layer* L) {
  const int d = L->desc.d_model;
  int dev = 0, max_smem = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  const int gm = L->desc.gate_mode;
  int stages = 16;
  while (stages > 1 && ffn_smem_bytes(d, stages, gm) > (size_t)max_smem) --stages;
  if (ffn_smem_bytes(d, stages, gm) > (size_t)max_smem) return cudaErrorInvalidValue;
  L->ffn_stages = L->ffn_stages_max = stages;
  L->ffn_smem = ffn_smem_bytes(d, stages, gm);
  return cudaFuncSetAttribute(ffn_kernel_for(gm), cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)max_smem);
}

static FfnArgs ffn_args(lif_layer* L, const __half* x, const int32_t* slots, const int32_t* n,
                        const int32_t* base, float* partial, int slots_len) {
  FfnArgs a;
  a.cache = (const __half*)L->desc.dev_cache;
  a.bias = L->bias;
  a.x = x;
  a.slots = slots;
  a.n = n;
  a.base = base;
  a.y_partial = partial;
  a.status = L->counts + LIF_CNT_STATUS;
  a.d = L->desc.d_model;
  a.stages = L->ffn_stages;
  a.slots_len = slots_len;
  a.act = L->desc.activation;
  a.act_thr = L->desc.activation_threshold;
  a.gate_val = L->gate_val;
  a.pointers = L->pointers;
  a.rows = L->desc.capacity;
  a.wait_polls = L->wait_polls;
  return a;
}

cudaError_t launch_ffn(lif_layer* L, const __half* x, const int32_t* slots, const int32_t* n,
                       const int32_t* base, float* y, bool accumulate, cudaStream_t st,
                       cudaEvent_t* ev) {
  const lif_layer_desc& D = L->desc;
  const int d = D.d_model;
  if (L->fb_ok && !accumulate) {   // several streams: tensor-core contraction over the rows
    if (ev) tm_record(ev[7], st);
    cudaError_t e = launch_ffn_batched(L, x, slots, n, base, y, st);
    if (ev) {
      tm_record(ev[8], st);
      tm_record(ev[9], st);
    }
    return e;
  }
  if (ev) tm_record(ev[7], st);
  for (int s = 0; s < D.n_streams; ++s) {
    // a caller's slot list may be shorter than d_ff: never read it before n is known
    FfnArgs a = ffn_args(L, x + (size_t)s * d, slots, n, base, L->y_partial,
                         slots && (slots == L->active_slots || slots == L->hit_slots) ? D.d_ff : 0);
    if (a.gate_val) a.gate_val += (size_t)s * D.d_ff;
    cudaError_t e = launch_k(ffn_kernel_for(D.gate_mode), dim3(L->ffn_grid), dim3(kThreads),
                             L->ffn_smem, st, L->use_pdl, a);
    if (e != cudaSuccess) return e;
    if (ev && s == D.n_streams - 1) tm_record(ev[8], st);
    e = launch_k(ffn_reduce_kernel, dim3((d / 4 + kSumCols - 1) / kSumCols), dim3(kSumThreads), 0, st, L->use_pdl,
                 (const float*)L->y_partial, n, (const float*)nullptr, (const int32_t*)nullptr,
                 L->ffn_grid, (const __half*)D.dev_bias_down, d, y + (size_t)s * d, d,
                 accumulate ? 1 : 0, D.capacity, (int*)nullptr);
    if (e != cudaSuccess) return e;
  }
  if (ev) tm_record(ev[9], st);
  return cudaSuccess;
}

cudaError_t launch_one(lif_layer* L, int kernel, const __half* x, float* y, cudaStream_t st) {
  const lif_layer_desc& D = L->desc;
  const int d = D.d_model;
  const int32_t* cnt = L->counts;
  float* p0 = L->y_partial;
  float* p1 = L->y_partial + (size_t)L->ffn_grid * d;
  FfnArgs a;
  switch (kernel) {
    case LIF_KERNEL_FFN_ACTIVE:
      a = ffn_args(L, x, L->active_slots, cnt + LIF_CNT_N_ACTIVE, nullptr, p0, D.d_ff);
      break;
    case LIF_KERNEL_FFN_HITS:
      a = ffn_args(L, x, L->hit_slots, cnt + LIF_CNT_N_HITS, nullptr, p0, D.d_ff);
      break;
    case LIF_KERNEL_FFN_NEW:
      a = D.append_first
              ? ffn_args(L, x, L->load_slots, cnt + LIF_CNT_N_LOAD, nullptr, p1, 0)
              : ffn_args(L, x, nullptr, cnt + LIF_CNT_N_LOAD, cnt + LIF_CNT_NUM_KEPT, p1, 0);
      break;
    case LIF_KERNEL_FFN_CACHE:      // every cached row: rows [0, num_used) after a completed step
      a = ffn_args(L, x, nullptr, cnt + LIF_CNT_NUM_USED, nullptr, p0, 0);
      break;
    case LIF_KERNEL_FFN_SUM:
      return launch_k(ffn_reduce_kernel, dim3((d / 4 + kSumCols - 1) / kSumCols), dim3(kSumThreads), 0, st,
                      L->use_pdl, (const float*)p0, cnt + LIF_CNT_N_HITS, (const float*)p1,
                      cnt + LIF_CNT_N_LOAD, L->ffn_grid, (const __half*)D.dev_bias_down, d, y, d, 0,
                      D.capacity, (int*)nullptr);
    default:
      return cudaErrorInvalidValue;
  }
  return launch_k(ffn_kernel_for(D.gate_mode), dim3(L->ffn_grid), dim3(kThreads), L->ffn_smem, st,
                  L->use_pdl, a);
}

cudaError_t launch_partial_sum(lif_layer* L, const float* partial, const int32_t* n,
                               int partitions, int width, float* y, cudaStream_t st) {
  return launch_k(ffn_reduce_kernel, dim3((width / 4 + kSumCols - 1) / kSumCols),
                  dim3(kSumThreads), 0, st, L->use_pdl, partial, n, (const float*)nullptr,
                  (const int32_t*)nullptr, partitions, (const __half*)L->desc.dev_bias_down,
                  L->desc.d_model, y, width, 0, L->desc.capacity, (int*)nullptr);
}

// Fetch + FFN of a single-stream decode step.  The critical chain stays on `st` with dependent
// launches: fetch -> FFN over the rows just brought in -> sum.  The FFN over the rows that
// were already cached does not depend on the fetch and runs on `side` meanwhile (forked after
// the row moves, joined before the sum).
cudaError_t launch_fetch_and_ffn_split(lif_layer* L, const __half* x, float* y, cudaStream_t st,
                                       cudaStream_t side, cudaEvent_t* ev, bool moves_aside) {
  const lif_layer_desc& D = L->desc;
  const int d = D.d_model;
  const int32_t* cnt = L->counts;
  float* p0 = L->y_partial;
  float* p1 = L->y_partial + (size_t)L->ffn_grid * d;
  const bool fork = side != st;
  cudaError_t e;
  if (fork) {
    if ((e = cudaEventRecord(L->ev_plan, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(side, L->ev_plan, 0)) != cudaSuccess) return e;
  }
  // append_first with a second stream: the row moves run there, ahead of the cached rows' FFN
  if (moves_aside && (e = launch_moves(L, side, ev)) != cudaSuccess) return e;
  FfnArgs hit = D.ffn_mode == 0
                    ? ffn_args(L, x, L->hit_slots, cnt + LIF_CNT_N_HITS, nullptr, p0, D.d_ff)
                    : ffn_args(L, x, nullptr, cnt + LIF_CNT_NUM_KEPT, nullptr, p0, 0);
  if (ev) tm_record(ev[7], side);
  e = launch_k(ffn_kernel_for(D.gate_mode), dim3(L->ffn_grid), dim3(kThreads), L->ffn_smem, side,
               fork ? 0 : L->use_pdl, hit);
  if (e != cudaSuccess) return e;
  if (ev) tm_record(ev[8], side);
  if (fork && (e = cudaEventRecord(L->ev_fetch, side)) != cudaSuccess) return e;
  if (ev) tm_record(ev[5], st);
  // the new rows: consecutive from num_kept, or (append_first) wherever load_slots says
  FfnArgs miss = D.append_first
                     ? ffn_args(L, x, L->load_slots, cnt + LIF_CNT_N_LOAD, nullptr, p1, 0)
                     : ffn_args(L, x, nullptr, cnt + LIF_CNT_N_LOAD, cnt + LIF_CNT_NUM_KEPT, p1, 0);
  if (L->fused_fetch && fetch_ffn_supported(L)) {
    // one kernel brings the new rows in and adds their FFN terms (CTA partials in p1)
    if ((e = launch_fetch_ffn(L, x, p1, st, L->watch_chain ? kEarlyWatch : (moves_aside ? kEarlyMask : kEarlyLists))) != cudaSuccess) return e;
    if (ev) tm_record(ev[6], st);
  } else {
    e = L->watch_chain ? launch_fetch_early(L, st, kEarlyWatch) : launch_fetch(L, st);
    if (e != cudaSuccess) return e;
    if (ev) tm_record(ev[6], st);
    e = launch_k(ffn_kernel_for(D.gate_mode), dim3(L->ffn_grid), dim3(kThreads), L->ffn_smem, st,
                 L->use_pdl, miss);
    if (e != cudaSuccess) return e;
  }
  if (fork && (e = cudaStreamWaitEvent(st, L->ev_fetch, 0)) != cudaSuccess) return e;
  e = launch_k(ffn_reduce_kernel, dim3((d / 4 + kSumCols - 1) / kSumCols), dim3(kSumThreads), 0,
               st, L->use_pdl, (const float*)p0, hit.n, (const float*)p1, miss.n, L->ffn_grid,
               (const __half*)D.dev_bias_down, d, y, d, 0, D.capacity,
               (int*)(L->counts + CNT_PREDICTOR_RUN));
  if (ev) tm_record(ev[9], st);
  return e;
}

}  // namespace lif

// ---------------------------------------------------------------------------------------------
// lif_sparse_ffn_static: the same two kernels, for callers that cannot provide a workspace.
// The CTA partials go to a fixed array in the library's own device image instead of
// caller-allocated memory.  Nothing here allocates: no cudaMalloc/cudaFree, no events, no
// library call that allocates.
// ---------------------------------------------------------------------------------------------
namespace lif {
namespace {

constexpr int kStaticFloats = 512 * 1024;   // 2 MiB of partials, resident on every device
constexpr int kStaticMaxDevices = 64;

struct StaticScratch {
  int32_t status;                // sticky lif_status of the kernels (bad row, wait that ran out);
                                 // read and cleared by lif_sparse_ffn_static_status
  int32_t pad[63];
  float partial[kStaticFloats];  // [ctas][d_model]
};
static __device__ __align__(256) StaticScratch g_static_scratch;

// Per-device set-up, done by the first call on that device: the device address of the
// scratch array (the symbol's name is only a host-side handle, never a device pointer), the
// shared-memory opt-in of the kernel on that device, and the launch shape limits.
struct StaticDevice {
  bool ready;
  StaticScratch* scratch;
  int n_sm, max_smem;
};
StaticDevice g_static_dev[kStaticMaxDevices];
std::mutex g_static_mutex;

}  // namespace
}  // namespace lif

namespace lif {
namespace {
// First use on the current device: resolve the scratch array's device address and opt the
// kernel in to large shared memory.  Returns nullptr (and leaves `err`) on failure.
StaticDevice* static_device(lif_status* err) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    *err = LIF_ERR_CUDA;
    return nullptr;
  }
  if (dev < 0 || dev >= kStaticMaxDevices) {
    *err = LIF_ERR_STATE;
    return nullptr;
  }
  StaticDevice& sd = g_static_dev[dev];
  std::lock_guard<std::mutex> setup_lock(g_static_mutex);   // first calls from several threads
  if (!sd.ready) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) !=
            cudaSuccess ||
        cudaFuncSetAttribute(sparse_ffn_kernel<LIF_GATE_NONE>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sd.max_smem) != cudaSuccess) {
      cudaGetLastError();
      *err = LIF_ERR_CUDA;
      return nullptr;
    }
    sd.scratch = static_cast<StaticScratch*>(p);
    sd.ready = true;
  }
  return &sd;
}
}  // namespace
}  // namespace lif

extern "C" lif_status lif_sparse_ffn_static_status(int32_t* host_status, int32_t clear) {
  using namespace lif;
  if (!host_status) return LIF_ERR_INVALID_ARG;
  lif_status err = LIF_OK;
  StaticDevice* sd = static_device(&err);
  if (!sd) return err;
  bool ok = cudaDeviceSynchronize() == cudaSuccess &&
            cudaMemcpy(host_status, &sd->scratch->status, sizeof(int32_t),
                       cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && clear) ok = cudaMemset(&sd->scratch->status, 0, sizeof(int32_t)) == cudaSuccess;
  if (!ok) cudaGetLastError();
  return ok ? LIF_OK : LIF_ERR_CUDA;
}

extern "C" lif_status lif_sparse_ffn_static(const void* dev_matrix, int32_t n_rows,
                                            const void* dev_bias, const void* dev_x,
                                            const int32_t* dev_slots, const int32_t* dev_n_slots,
                                            const void* dev_bias_down, float* dev_y,
                                            int32_t d_model, void* stream) {
  using namespace lif;
  if (!dev_matrix || !dev_bias || !dev_x || !dev_n_slots || !dev_y || n_rows < 1)
    return LIF_ERR_INVALID_ARG;
  // the scratch holds at least 64 CTA partials of this width
  if (d_model < 8 || d_model % 8 || d_model > LIF_STATIC_MAX_D_MODEL) return LIF_ERR_INVALID_ARG;
  auto mis = [](const void* p, size_t a) { return ((uintptr_t)p % a) != 0; };
  if (mis(dev_matrix, 16) || mis(dev_x, 16) || mis(dev_y, 16) || mis(dev_bias, 2) ||
      mis(dev_n_slots, 4) || (dev_slots && mis(dev_slots, 4)) ||
      (dev_bias_down && mis(dev_bias_down, 8)))
    return LIF_ERR_ALIGNMENT;

  lif_status err = LIF_OK;
  StaticDevice* sdp = static_device(&err);
  if (!sdp) return err;
  StaticDevice& sd = *sdp;

  int stages = 16;
  while (stages > 1 && ffn_smem_bytes(d_model, stages) > (size_t)sd.max_smem) --stages;
  if (ffn_smem_bytes(d_model, stages) > (size_t)sd.max_smem) return LIF_ERR_INVALID_ARG;
  int grid = kStaticFloats / d_model;
  if (grid > sd.n_sm) grid = sd.n_sm;

  cudaStream_t st = (cudaStream_t)stream;
  FfnArgs a;
  a.cache = (const __half*)dev_matrix;
  a.bias = (const __half*)dev_bias;
  a.x = (const __half*)dev_x;
  a.slots = dev_slots;
  a.n = dev_n_slots;
  a.base = nullptr;
  a.y_partial = sd.scratch->partial;
  a.status = &sd.scratch->status;
  a.d = d_model;
  a.stages = stages;
  a.slots_len = 0;
  a.act = LIF_ACT_RELU;
  a.act_thr = 0.f;
  a.gate_val = nullptr;
  a.pointers = nullptr;
  a.rows = n_rows;
  a.wait_polls = kWaitLimit;
  sparse_ffn_kernel<LIF_GATE_NONE><<<grid, kThreads, ffn_smem_bytes(d_model, stages), st>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LIF_ERR_CUDA;
  ffn_reduce_kernel<<<(d_model / 4 + kSumCols - 1) / kSumCols, kSumThreads, 0, st>>>(
      sd.scratch->partial, dev_n_slots, nullptr, nullptr, grid, (const __half*)dev_bias_down,
      d_model, dev_y, d_model, 0, n_rows, (int*)nullptr);
  return cudaGetLastError() == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}
