// Sparse FFN for several decode streams sharing one layer (Section 3.3 item 3 applied to S
// inputs at once): over the gathered rows the computation is a dense contraction,
//   H[q][s] = relu(<M[slot_q, :d], x[s]> + bias[slot_q])        (up halves,   K = d_model)
//   Y[s][m] = b_down[m] + sum_q H[q][s] * M[slot_q, d + m]       (down halves, K = rows)
// so it runs on tensor cores (mma.sync m16n8k16, fp16 operands, fp32 accumulate) while every
// bundle half is still read from HBM exactly once:
//   phase A: CTAs own rows; the up halves stream through a ring of shared-memory stages (one
//            bulk copy per half row), x (S x d, fp16) stays in shared memory as the A operand,
//            the rows are the B operand; the 8 warps split K and fold through shared memory.
//   phase B: CTAs own (row partition, column part); the down halves of the part stream through
//            the ring, 16 rows per MMA k-step; H (split into fp16 high + low parts, so the
//            product keeps fp32 accuracy) is the B operand; each warp keeps its column tiles'
//            accumulators in registers for the whole kernel.
// Partition partials are added in a fixed order by the partial-sum kernel.  Bound: HBM.
#include "lif_internal.cuh"

namespace lif {
namespace {

constexpr int kPad = 16;                  // bytes added to every shared row: conflict-free ldmatrix
constexpr unsigned kWaitLimitB = 1u << 22;
constexpr int kGroupA = 4;                // rows per MMA in phase A (N = 8, half used)
constexpr int kMaxTilesPerWarp = 28;      // 16-column tiles per warp in phase B

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
  for (unsigned i = 0; i < kWaitLimitB; ++i) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes,
                                         uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}

struct BatchedArgs {
  const __half* cache;
  const __half* bias;
  const __half* x;        // [S][d]
  const int32_t* slots;   // or nullptr: rows base .. base + n
  const int32_t* n;
  const int32_t* base;
  float* H;               // [n][8] fp32, position-indexed
  float* y_partial;       // [partitions][S][d]
  int32_t* status;
  int d, S, stages, parts, partitions, cols_per_part;
};

__device__ __forceinline__ int row_slot(const BatchedArgs& a, int q, int base) {
  return a.slots ? a.slots[q] : base + q;
}

// ---- phase A: H = relu(Up . X^T + bias) ------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1) ffn_batched_up_kernel(BatchedArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = a.d;
  const unsigned half_bytes = 2u * d;
  const unsigned pitch = half_bytes + kPad;
  const int stages = a.stages;               // multiple of kGroupA, two groups or more
  unsigned char* xs = smem;                                  // [8][pitch]
  unsigned char* rows = xs + 8 * (size_t)pitch;              // [stages][pitch]
  uint64_t* bars = reinterpret_cast<uint64_t*>(rows + (size_t)stages * pitch);
  float* bias_s = reinterpret_cast<float*>(bars + stages);   // [stages]
  float* red = bias_s + stages;                              // [8 warps][32 lanes][2]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();
  const int n = *a.n;
  if (cta >= n) return;
  const int base = a.base ? *a.base : 0;
  const int my_cnt = (n - cta + G - 1) / G;   // rows q = cta + i * G
  __syncthreads();

  // first copies in flight, then x into shared memory (streams beyond S are zero)
  if (tid < stages && tid < my_cnt) {
    const int slot = row_slot(a, cta + tid * G, base);
    mbar_expect_tx(bars + tid, half_bytes);
    bulk_g2s(rows + (size_t)tid * pitch, a.cache + (size_t)slot * 2 * d, half_bytes, bars + tid);
    bias_s[tid] = __half2float(a.bias[slot]);
  }
  {
    const int vec = d >> 3;
    for (int i = tid; i < 8 * vec; i += kThreads) {
      const int s = i / vec, c = i % vec;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (s < a.S) v = reinterpret_cast<const uint4*>(a.x + (size_t)s * d)[c];
      *reinterpret_cast<uint4*>(xs + (size_t)s * pitch + (size_t)c * 16) = v;
    }
  }
  __syncthreads();

  const int ksteps = d >> 4;
  const int kper = (ksteps + 7) >> 3;
  const int k_begin = warp * kper, k_end = min(ksteps, k_begin + kper);
  const int gq = lane >> 2, tq = lane & 3;          // fragment coordinates
  const unsigned char* xa = xs + (size_t)gq * pitch + tq * 4;           // A: stream gq
  int timed_out = 0;
  const int n_groups = (my_cnt + kGroupA - 1) / kGroupA;
  const int groups_in_ring = stages / kGroupA;
  for (int g = 0; g < n_groups; ++g) {
    const int st0 = (g % groups_in_ring) * kGroupA;
    const unsigned parity = (unsigned)(g / groups_in_ring) & 1u;
    const int valid = min(kGroupA, my_cnt - g * kGroupA);
    for (int i = 0; i < valid; ++i)
      if (!mbar_wait(bars + st0 + i, parity)) timed_out = 1;
    // D[stream][row] over this warp's K slice; B column = row gq of the group (gq < 4)
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    const unsigned char* rb = rows + (size_t)(st0 + (gq & 3)) * pitch + tq * 4;
    const bool brow = gq < kGroupA;
#pragma unroll 4
    for (int k = k_begin; k < k_end; ++k) {
      uint32_t af[4];
      af[0] = *reinterpret_cast<const uint32_t*>(xa + k * 32);
      af[1] = 0u;
      af[2] = *reinterpret_cast<const uint32_t*>(xa + k * 32 + 16);
      af[3] = 0u;
      uint32_t b0 = 0u, b1 = 0u;
      if (brow) {
        b0 = *reinterpret_cast<const uint32_t*>(rb + k * 32);
        b1 = *reinterpret_cast<const uint32_t*>(rb + k * 32 + 16);
      }
      mma16816(c, af, b0, b1);
    }
    // c[0], c[1] = (stream gq, rows 2*tq, 2*tq + 1); fold the 8 warps
    red[(warp * 32 + lane) * 2] = c[0];
    red[(warp * 32 + lane) * 2 + 1] = c[1];
    if (__syncthreads_or(timed_out)) {
      if (tid == 0) {
        atomicCAS(a.status, LIF_OK, LIF_ERR_TIMEOUT);
        for (int i = 0; i < valid; ++i) mbar_wait(bars + st0 + i, parity);
      }
      __syncthreads();
      return;
    }
    if (tid < 8 * kGroupA) {
      const int s = tid >> 2, r = tid & 3;          // stream, row in group
      if (r < valid) {
        const int src_lane = s * 4 + (r >> 1);
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[(w * 32 + src_lane) * 2 + (r & 1)];
        v = fmaxf(v + bias_s[st0 + r], 0.f);
        const int q = cta + (g * kGroupA + r) * G;
        a.H[(size_t)q * 8 + s] = v;
      }
    }
    __syncthreads();                                 // stages st0.. and bias_s are free
    // refill with the rows of group g + groups_in_ring
    if (tid < kGroupA) {
      const int i = (g + groups_in_ring) * kGroupA + tid;
      if (i < my_cnt) {
        const int slot = row_slot(a, cta + i * G, base);
        mbar_expect_tx(bars + st0 + tid, half_bytes);
        bulk_g2s(rows + (size_t)(st0 + tid) * pitch, a.cache + (size_t)slot * 2 * d, half_bytes,
                 bars + st0 + tid);
        bias_s[st0 + tid] = __half2float(a.bias[slot]);
      }
    }
  }
}

// ---- phase B: Y^T[cols of part] += Down^T . H over this partition's rows ---------------------
__global__ void __launch_bounds__(kThreads, 1) ffn_batched_down_kernel(BatchedArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = a.d;
  const int part = blockIdx.x % a.parts, prt = blockIdx.x / a.parts;
  const int col0 = part * a.cols_per_part;
  const int ncols = min(a.cols_per_part, d - col0);
  const unsigned seg_bytes = 2u * ncols;
  const unsigned pitch = 2u * a.cols_per_part + kPad;
  const int stages = a.stages;                   // 32: two groups of 16 rows
  unsigned char* rows = smem;                                          // [stages][pitch]
  uint64_t* bars = reinterpret_cast<uint64_t*>(rows + (size_t)stages * pitch);
  __half* h_hi = reinterpret_cast<__half*>(bars + stages);             // [8][16]
  __half* h_lo = h_hi + 128;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // zero the row buffers once: padded k-steps multiply by H = 0 and need finite operands
  for (size_t i = (size_t)tid * 16; i < (size_t)stages * pitch; i += kThreads * 16)
    *reinterpret_cast<uint4*>(rows + i) = make_uint4(0, 0, 0, 0);
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  pdl_wait();
  pdl_trigger();
  const int n = *a.n;
  const int base = a.base ? *a.base : 0;
  const int P = a.partitions;
  const int my_cnt = prt < n ? (n - prt + P - 1) / P : 0;       // rows q = prt + i * P
  const size_t col_off = (size_t)d + col0;

  if (tid < stages && tid < my_cnt) {
    const int slot = row_slot(a, prt + tid * P, base);
    mbar_expect_tx(bars + tid, seg_bytes);
    bulk_g2s(rows + (size_t)tid * pitch, a.cache + (size_t)slot * 2 * d + col_off, seg_bytes,
             bars + tid);
  }

  const int tiles = (ncols + 15) >> 4;
  float acc[kMaxTilesPerWarp][4];
#pragma unroll
  for (int t = 0; t < kMaxTilesPerWarp; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;

  // H of the next group, prefetched: thread (k = tid / 8, s = tid % 8) for tid < 128
  const int hk = tid >> 3, hs = tid & 7;
  float h_next = 0.f;
  if (tid < 128 && hk < my_cnt) h_next = a.H[(size_t)(prt + hk * P) * 8 + hs];

  int timed_out = 0;
  const int n_groups = (my_cnt + 15) >> 4;
  const int gq = lane >> 2, tq = lane & 3;
  for (int g = 0; g < n_groups; ++g) {
    const int st0 = (g & 1) * 16;
    const unsigned parity = (unsigned)(g >> 1) & 1u;
    const int valid = min(16, my_cnt - g * 16);
    if (tid < 128) {
      const float h = hk < valid ? h_next : 0.f;
      const __half hi = __float2half_rn(h);
      h_hi[hs * 16 + hk] = hi;
      h_lo[hs * 16 + hk] = __float2half_rn(h - __half2float(hi));
      const int i = (g + 1) * 16 + hk;
      h_next = i < my_cnt ? a.H[(size_t)(prt + i * P) * 8 + hs] : 0.f;
    }
    for (int i = 0; i < valid; ++i)
      if (!mbar_wait(bars + st0 + i, parity)) timed_out = 1;
    if (__syncthreads_or(timed_out)) {
      if (tid == 0) {
        atomicCAS(a.status, LIF_OK, LIF_ERR_TIMEOUT);
        for (int i = 0; i < valid; ++i) mbar_wait(bars + st0 + i, parity);
      }
      __syncthreads();
      return;
    }
    // B fragments: H[k][n], k = 2*tq (+8), n = gq
    const uint32_t bh0 = *reinterpret_cast<const uint32_t*>(h_hi + gq * 16 + tq * 2);
    const uint32_t bh1 = *reinterpret_cast<const uint32_t*>(h_hi + gq * 16 + tq * 2 + 8);
    const uint32_t bl0 = *reinterpret_cast<const uint32_t*>(h_lo + gq * 16 + tq * 2);
    const uint32_t bl1 = *reinterpret_cast<const uint32_t*>(h_lo + gq * 16 + tq * 2 + 8);
    // A fragments: Down^T tile (16 columns x 16 rows), read transposed from the row-major stage
    const unsigned char* abase =
        rows + (size_t)(st0 + (lane & 7) + ((lane >> 4) << 3)) * pitch + ((lane >> 3) & 1) * 16;
#pragma unroll
    for (int t = 0; t < kMaxTilesPerWarp; ++t) {
      const int tile = warp + t * 8;
      if (tile < tiles) {
        uint32_t af[4];
        ldmatrix_x4_trans(af, abase + tile * 32);
        mma16816(acc[t], af, bh0, bh1);
        mma16816(acc[t], af, bl0, bl1);
      }
    }
    __syncthreads();                               // stages of this group and h_hi/h_lo are free
    if (tid < 16) {
      const int i = (g + 2) * 16 + tid;
      if (i < my_cnt) {
        const int slot = row_slot(a, prt + i * P, base);
        mbar_expect_tx(bars + st0 + tid, seg_bytes);
        bulk_g2s(rows + (size_t)(st0 + tid) * pitch, a.cache + (size_t)slot * 2 * d + col_off,
                 seg_bytes, bars + st0 + tid);
      }
    }
  }
  // epilogue: acc[t] = (column gq (+8) of the tile, streams 2*tq, 2*tq + 1)
  float* out = a.y_partial + (size_t)prt * a.S * d;
#pragma unroll
  for (int t = 0; t < kMaxTilesPerWarp; ++t) {
    const int tile = warp + t * 8;
    if (tile < tiles) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int m = tile * 16 + gq + (e >> 1) * 8;
        const int s = tq * 2 + (e & 1);
        if (m < ncols && s < a.S) out[(size_t)s * d + col0 + m] = acc[t][e];
      }
    }
  }
}

// y[s][m] = b_down[m] + sum_p y_partial[p][s][m], p ascending
__global__ void __launch_bounds__(kThreads)
ffn_batched_sum_kernel(const float* __restrict__ y_partial, int partitions,
                       const __half* __restrict__ b_down, float* __restrict__ y, int d, int S) {
  pdl_wait();
  pdl_trigger();
  const size_t total4 = (size_t)S * d / 4;
  const size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= total4) return;
  const int m = (int)((i * 4) % d);
  float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
  if (b_down) {
    const __half2* b = reinterpret_cast<const __half2*>(b_down + m);
    const float2 lo = __half22float2(b[0]), hi = __half22float2(b[1]);
    t = make_float4(lo.x, lo.y, hi.x, hi.y);
  }
#pragma unroll 8
  for (int p = 0; p < partitions; ++p) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(y_partial + (size_t)p * S * d) + i);
    t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
  }
  reinterpret_cast<float4*>(y)[i] = t;
}

size_t up_smem(int d, int stages) {
  const size_t pitch = 2 * (size_t)d + kPad;
  return (8 + stages) * pitch + stages * 8 + stages * 4 + 8 * 32 * 2 * 4 + 16;
}
size_t down_smem(int cols_per_part, int stages) {
  return stages * (2 * (size_t)cols_per_part + kPad) + stages * 8 + 2 * 128 * 2 + 16;
}

}  // namespace

bool ffn_batched_supported(const lif_layer_desc& D) { return D.n_streams > 1 && D.d_model % 16 == 0; }

cudaError_t ffn_batched_configure(lif_layer* L) {
  const lif_layer_desc& D = L->desc;
  L->fb_ok = 0;
  if (!ffn_batched_supported(D)) return cudaSuccess;
  int dev = 0, max_smem = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  const int d = D.d_model;
  int st = 16;                                     // phase A: multiple of kGroupA, >= 2 groups
  while (st > 2 * kGroupA && up_smem(d, st) > (size_t)max_smem) st -= kGroupA;
  if (up_smem(d, st) > (size_t)max_smem) return cudaSuccess;   // fall back to the per-stream path
  const int tiles = d / 16;
  int parts = 1;
  while ((tiles + parts - 1) / parts > 8 * kMaxTilesPerWarp ||
         down_smem((tiles + parts - 1) / parts * 16, 32) > (size_t)max_smem)
    ++parts;
  L->fb_up_stages = st;
  L->fb_up_smem = up_smem(d, st);
  L->fb_parts = parts;
  L->fb_cols = (tiles + parts - 1) / parts * 16;
  L->fb_partitions = L->n_sm / parts > 0 ? L->n_sm / parts : 1;
  if (L->fb_partitions > kBatchedMaxPartitions) L->fb_partitions = kBatchedMaxPartitions;
  L->fb_down_smem = down_smem(L->fb_cols, 32);
  e = cudaFuncSetAttribute(ffn_batched_up_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           max_smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(ffn_batched_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           max_smem);
  if (e != cudaSuccess) return e;
  L->fb_ok = 1;
  return cudaSuccess;
}

cudaError_t launch_ffn_batched(lif_layer* L, const __half* x, const int32_t* slots,
                               const int32_t* n, const int32_t* base, float* y, cudaStream_t st) {
  const lif_layer_desc& D = L->desc;
  BatchedArgs a;
  a.cache = (const __half*)D.dev_cache;
  a.bias = L->bias;
  a.x = x;
  a.slots = slots;
  a.n = n;
  a.base = base;
  a.H = L->h_rows;
  a.y_partial = L->y_partial;
  a.status = L->counts + LIF_CNT_STATUS;
  a.d = D.d_model;
  a.S = D.n_streams;
  a.parts = L->fb_parts;
  a.partitions = L->fb_partitions;
  a.cols_per_part = L->fb_cols;
  a.stages = L->fb_up_stages;
  cudaError_t e = launch_k(ffn_batched_up_kernel, dim3(L->n_sm), dim3(kThreads), L->fb_up_smem, st,
                           L->use_pdl, a);
  if (e != cudaSuccess) return e;
  a.stages = 32;
  e = launch_k(ffn_batched_down_kernel, dim3(L->fb_parts * L->fb_partitions), dim3(kThreads),
               L->fb_down_smem, st, L->use_pdl, a);
  if (e != cudaSuccess) return e;
  const size_t total4 = (size_t)D.n_streams * D.d_model / 4;
  return launch_k(ffn_batched_sum_kernel, dim3((unsigned)((total4 + kThreads - 1) / kThreads)),
                  dim3(kThreads), 0, st, L->use_pdl, (const float*)L->y_partial, L->fb_partitions,
                  (const __half*)D.dev_bias_down, y, D.d_model, D.n_streams);
}

}  // namespace lif
