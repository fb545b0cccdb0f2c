// Sparse FFN over cached row-column bundles (Section 3.3 item 3):
//   y = b_down + sum_q relu(<M[slot_q, :d], x> + bias[slot_q]) * M[slot_q, d:]
// A bundle is one contiguous 4*d_model-byte row (Section 3.2), so the unit of HBM traffic is
// one bulk asynchronous copy (TMA, cp.async.bulk) of a whole row into shared memory.  Each
// CTA owns rows q = cta, cta + G, ...; it issues the copies for all its rows up front (up to
// `stages` in flight), and as each row's mbarrier completes the 256 threads dot the up half
// with x (16-byte shared loads, warp-shuffle + 8-way shared reduction), apply bias + ReLU, and
// axpy the down half into fp32 register accumulators.  Rows whose ReLU is zero skip the axpy.
// CTA partials go to a [G][d] fp32 scratch; a second kernel adds them in CTA order, so the
// result does not depend on scheduling.  Bound: HBM bandwidth, 4*d_model bytes per row.
#include "lif_internal.cuh"

namespace lif {
namespace {

constexpr int kMaxChunks = 4;            // 8-column chunks per thread: d_model <= 8192
constexpr unsigned kWaitLimit = 1u << 22;

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
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the barrier did not complete within kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity) {
  for (unsigned i = 0; i < kWaitLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes,
                                         uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

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
};

__global__ void __launch_bounds__(kThreads, 1) sparse_ffn_kernel(FfnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = a.d;
  const unsigned row_bytes = 4u * d;
  const int stages = a.stages;
  // shared layout: rows[stages][row_bytes] | x[d] fp16 | bars[stages] | part[stages][8] |
  //                h[stages] | slot[stages]
  unsigned char* rows = smem;
  __half* xs = reinterpret_cast<__half*>(rows + (size_t)stages * row_bytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(xs) +
                                               (((size_t)d * 2 + 15) & ~(size_t)15));
  float* part = reinterpret_cast<float*>(bars + stages);
  float* hs = part + stages * 8;
  int* slot_s = reinterpret_cast<int*>(hs + stages);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const int n = *a.n;
  if (cta >= n) return;                       // the reduction only reads min(G, n) partials
  const int base = a.base ? *a.base : 0;
  const int my_cnt = (n - cta + G - 1) / G;
  const int nvec = d >> 3;                    // 16-byte chunks per half row

  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  float acc[kMaxChunks][8];
#pragma unroll
  for (int c = 0; c < kMaxChunks; ++c)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[c][e] = 0.f;

  unsigned parity = 0;
  int timed_out = 0;
  for (int r0 = 0; r0 < my_cnt; r0 += stages) {
    const int rc = min(stages, my_cnt - r0);
    if (tid == 0) {
      for (int i = 0; i < rc; ++i) {
        const int q = cta + (r0 + i) * G;
        const int slot = a.slots ? a.slots[q] : base + q;
        slot_s[i] = slot;
        mbar_expect_tx(bars + i, row_bytes);
        bulk_g2s(rows + (size_t)i * row_bytes, a.cache + (size_t)slot * 2 * d, row_bytes,
                 bars + i);
      }
    }
    if (r0 == 0) {
      const uint4* xg = reinterpret_cast<const uint4*>(a.x);
      for (int c = tid; c < nvec; c += kThreads) reinterpret_cast<uint4*>(xs)[c] = xg[c];
      __syncthreads();
    }
    // up projection: partial dot products as rows land
    for (int i = 0; i < rc; ++i) {
      if (!mbar_wait(bars + i, parity)) timed_out = 1;
      const uint4* up = reinterpret_cast<const uint4*>(rows + (size_t)i * row_bytes);
      float p = 0.f;
      for (int c = tid; c < nvec; c += kThreads) {
        float uf[8], xf[8];
        unpack8(up[c], uf);
        unpack8(reinterpret_cast<const uint4*>(xs)[c], xf);
#pragma unroll
        for (int e = 0; e < 8; ++e) p = fmaf(uf[e], xf[e], p);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
      if (lane == 0) part[i * 8 + warp] = p;
    }
    if (__syncthreads_or(timed_out)) {
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
    if (tid < rc) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) v += part[tid * 8 + w];
      v += __half2float(a.bias[slot_s[tid]]);
      hs[tid] = fmaxf(v, 0.f);
    }
    __syncthreads();
    // down projection: y += h * down half
    for (int i = 0; i < rc; ++i) {
      const float h = hs[i];
      if (h == 0.f) continue;
      const uint4* down = reinterpret_cast<const uint4*>(rows + (size_t)i * row_bytes) + nvec;
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

// y[m] = (accumulate ? y[m] : b_down[m]) + sum_{g < min(G, n)} y_partial[g][m].  1024 threads =
// 32 float4 columns x 32 slices of g; each slice adds its partials in ascending g, then the
// slices are added in ascending order: a fixed summation order.
constexpr int kSumThreads = 1024;
__global__ void __launch_bounds__(kSumThreads)
ffn_reduce_kernel(const float* __restrict__ y_partial, int G, const int32_t* __restrict__ n,
                  const __half* __restrict__ b_down, float* __restrict__ y, int d,
                  int accumulate) {
  __shared__ float4 red[32][32];
  const int tid = threadIdx.x;
  const int c4 = tid & 31, gs = tid >> 5;
  const int col4 = blockIdx.x * 32 + c4;       // float4 column
  const int valid = min(G, *n);
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col4 * 4 < d) {
#pragma unroll 4
    for (int g = gs; g < valid; g += 32) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(y_partial + (size_t)g * d) + col4);
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
  }
  red[gs][c4] = s;
  __syncthreads();
  if (gs == 0 && col4 * 4 < d) {
    float4 t;
    if (accumulate) {
      t = reinterpret_cast<float4*>(y)[col4];
    } else if (b_down) {
      const __half2* b = reinterpret_cast<const __half2*>(b_down) + col4 * 2;
      const float2 lo = __half22float2(b[0]), hi = __half22float2(b[1]);
      t = make_float4(lo.x, lo.y, hi.x, hi.y);
    } else {
      t = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      t.x += red[k][c4].x; t.y += red[k][c4].y; t.z += red[k][c4].z; t.w += red[k][c4].w;
    }
    reinterpret_cast<float4*>(y)[col4] = t;
  }
}

size_t ffn_smem_bytes(int d, int stages) {
  size_t b = (size_t)stages * 4 * d;              // rows
  b += ((size_t)d * 2 + 15) & ~(size_t)15;        // x
  b += (size_t)stages * 8;                        // barriers
  b += (size_t)stages * 8 * 4 + (size_t)stages * 4 + (size_t)stages * 4;
  return b + 16;
}

}  // namespace

cudaError_t ffn_configure(lif_layer* L) {
  const int d = L->desc.d_model;
  int dev = 0, max_smem = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  int stages = 16;
  while (stages > 1 && ffn_smem_bytes(d, stages) > (size_t)max_smem) --stages;
  if (ffn_smem_bytes(d, stages) > (size_t)max_smem) return cudaErrorInvalidValue;
  L->ffn_stages = stages;
  L->ffn_smem = ffn_smem_bytes(d, stages);
  return cudaFuncSetAttribute(sparse_ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)max_smem);
}

cudaError_t launch_ffn(lif_layer* L, const __half* x, const int32_t* slots, const int32_t* n,
                       const int32_t* base, float* y, bool accumulate, cudaStream_t st,
                       cudaEvent_t* ev) {
  const lif_layer_desc& D = L->desc;
  const int d = D.d_model;
  if (ev) tm_record(ev[7], st);
  for (int s = 0; s < D.n_streams; ++s) {
    FfnArgs a;
    a.cache = (const __half*)D.dev_cache;
    a.bias = L->bias;
    a.x = x + (size_t)s * d;
    a.slots = slots;
    a.n = n;
    a.base = base;
    a.y_partial = L->y_partial;
    a.status = L->counts + LIF_CNT_STATUS;
    a.d = d;
    a.stages = L->ffn_stages;
    sparse_ffn_kernel<<<L->ffn_grid, kThreads, L->ffn_smem, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (ev && s == D.n_streams - 1) tm_record(ev[8], st);
    ffn_reduce_kernel<<<(d / 4 + 31) / 32, kSumThreads, 0, st>>>(
        L->y_partial, L->ffn_grid, n, (const __half*)D.dev_bias_down, y + (size_t)s * d, d,
        accumulate ? 1 : 0);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (ev) tm_record(ev[9], st);
  return cudaSuccess;
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
  int32_t status;                // sink for the kernel's timeout flag; cleared by every call
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

}  // namespace
}  // namespace lif

extern "C" lif_status lif_sparse_ffn_static(const void* dev_matrix, const void* dev_bias,
                                            const void* dev_x, const int32_t* dev_slots,
                                            const int32_t* dev_n_slots, const void* dev_bias_down,
                                            float* dev_y, int32_t d_model, void* stream) {
  using namespace lif;
  if (!dev_matrix || !dev_bias || !dev_x || !dev_n_slots || !dev_y) return LIF_ERR_INVALID_ARG;
  // the scratch holds at least 64 CTA partials of this width
  if (d_model < 8 || d_model % 8 || d_model > LIF_STATIC_MAX_D_MODEL) return LIF_ERR_INVALID_ARG;
  auto mis = [](const void* p, size_t a) { return ((uintptr_t)p % a) != 0; };
  if (mis(dev_matrix, 16) || mis(dev_x, 16) || mis(dev_y, 16) || mis(dev_bias, 2) ||
      mis(dev_n_slots, 4) || (dev_slots && mis(dev_slots, 4)) ||
      (dev_bias_down && mis(dev_bias_down, 8)))
    return LIF_ERR_ALIGNMENT;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LIF_ERR_CUDA;
  if (dev < 0 || dev >= kStaticMaxDevices) return LIF_ERR_STATE;
  StaticDevice& sd = g_static_dev[dev];
  if (!sd.ready) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sd.max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) !=
            cudaSuccess ||
        cudaFuncSetAttribute(sparse_ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             sd.max_smem) != cudaSuccess) {
      cudaGetLastError();
      return LIF_ERR_CUDA;
    }
    sd.scratch = static_cast<StaticScratch*>(p);
    sd.ready = true;
  }

  int stages = 16;
  while (stages > 1 && ffn_smem_bytes(d_model, stages) > (size_t)sd.max_smem) --stages;
  if (ffn_smem_bytes(d_model, stages) > (size_t)sd.max_smem) return LIF_ERR_INVALID_ARG;
  int grid = kStaticFloats / d_model;
  if (grid > sd.n_sm) grid = sd.n_sm;

  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(&sd.scratch->status, 0, sizeof(int32_t), st) != cudaSuccess) {
    cudaGetLastError();
    return LIF_ERR_CUDA;
  }
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
  sparse_ffn_kernel<<<grid, kThreads, ffn_smem_bytes(d_model, stages), st>>>(a);
  if (cudaGetLastError() != cudaSuccess) return LIF_ERR_CUDA;
  ffn_reduce_kernel<<<(d_model / 4 + 31) / 32, kSumThreads, 0, st>>>(
      sd.scratch->partial, grid, dev_n_slots, (const __half*)dev_bias_down, dev_y, d_model, 0);
  return cudaGetLastError() == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}
