// Bringing in new neurons (Section 3.3 item 2): gather the bundles of the newly needed
// neurons from the full store in mapped pinned host memory (standing in for flash) into
// their cache rows.  The kernel reads host memory directly: every warp instruction reads 512
// contiguous bytes of one bundle with 16-byte loads, and each thread keeps several loads in
// flight so the link sees enough outstanding requests.  Bound: host-link bandwidth.
#include "lif_internal.cuh"
#include "mask_compact.cuh"

namespace lif {
namespace {

constexpr int kFetchUnroll = 8;   // 16-byte loads in flight per thread

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
      if (v < row_vec) buf[i] = ld_stream16(src + v);
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

// Fetch and FFN of the new rows in one kernel (single stream, row = up | down of at most
// 32 KiB).  A CTA that brings a bundle in holds all of it in registers on its way from host
// memory to the cache row, so it also computes that neuron's term of the FFN
// (Section 3.3 item 3): h = act(<up, x> + bias) and partial += h * down.  The new rows then need
// no second pass over HBM and no kernel of their own after the slowest step of the layer.  Rows
// are dealt to CTAs in list order and each CTA adds its rows in that order, so the partials and
// their sum do not depend on scheduling.  Where the kernel ahead is the row-move kernel, the
// first bundle's host loads are issued before the dependency wait: the list and the counts were
// final before that kernel passed its own wait, while the cache rows may still be moving.
constexpr int kFusedChunks = 4;     // 8-column chunks per thread and half row: d_model <= 8192

// The predictor's entries of neurons to bring in, and where the run number lives.
struct EarlySource {
  const unsigned long long* entries;   // {bits, run}
  int nwords, word_bits;               // entries, and the consecutive neurons each one covers
  const int* predictor_run;            // number of the predictor run of this step
  const int32_t* counts;
};

struct FetchFfnArgs {
  const uint4* store;
  uint4* cache;
  const int32_t* load_ids;
  const int32_t* load_slots;
  const int32_t* counts;
  const __half* bias;        // per cache row
  const __half* x;
  const float* gate_val;     // resident gate: gate pre-activations by neuron id
  float* y_partial;          // [gridDim.x][d]
  int d, act;
  float act_thr;
  EarlySource early;         // what the mask-driven forms read ahead of the dependency wait
};

// How much of the kernel may run before its dependency wait:
//   kEarlyNone   nothing: the kernel ahead wrote the lists.
//   kEarlyLists  the lists were final before the kernel ahead passed its own wait (it is the
//                row-move kernel): count, ids and rows are read and the first bundle's host
//                loads issued ahead of the wait.
//   kEarlyMask   the kernel ahead is the window kernel, whose lists are not final yet, but the
//                predictor's entries of neurons to bring in are: the load list is exactly their
//                set bits in ascending order (the window kernel derives it from the same
//                state), so CTA c finds the id of its first bundle, the c-th set bit, itself
//                and its host loads travel while the window kernel runs.
//   kEarlyWatch  as kEarlyMask, but the kernel may be resident while the predictor still runs
//                and reads the entries as they arrive (see the kernel).
// In the last two forms nothing depends on what was read ahead of the wait: after it the count
// and the id are compared with the window kernel's list, and a CTA whose early reading differs
// (the window kernel refused the step, the entries were another run's) starts over from the list.
constexpr int kWatchPolls = 64;     // about 30 us of polling at most

// What a fetch kernel learned ahead of its dependency wait: the form it ended up in (kEarlyNone:
// the wait has been passed already; otherwise the caller still has to wait), the count of
// neurons to bring in (from the entries in kEarlyMask form, else the window kernel's) and, in
// kEarlyMask form, the id of the want-th of them (-1 if there are fewer).
struct EarlyPick {
  int mode, n, id;
};
template <int kEarlyT>
__device__ __forceinline__ EarlyPick early_pick(const EarlySource& src, int want, int* scan_sums,
                                                int* first_id) {
  const int tid = threadIdx.x;
  int kEarly = kEarlyT;
  // thread t owns a run of consecutive words of the mask of neurons to bring in
  const int wpt = (src.nwords + kThreads - 1) / kThreads;
  const int w0 = min(src.nwords, tid * wpt), w1 = min(src.nwords, w0 + wpt);
  uint32_t mw[4] = {0u, 0u, 0u, 0u};               // nwords <= 1024 in the mask-driven forms
  auto read_words = [&](int want_tag, bool check) {
    bool all_mine = true;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mw[i] = 0u;
      if (w0 + i < w1) {
        unsigned long long v;
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(src.entries + w0 + i)
                     : "memory");
        mw[i] = (uint32_t)v;
        all_mine = all_mine && (!check || (int)(v >> 32) == want_tag);
      }
    }
    return all_mine;
  };
  if (kEarlyT == kEarlyWatch) {
    // Resident while the predictor may still be running (all of its CTAs are: it released the
    // window kernel, which released this one, only after every one of them had started).  Every
    // mask word is stored together with the number of the predictor run that wrote it (one
    // 8-byte store), and that number was fixed before the run began, so each thread simply
    // re-reads its own words until all of them carry it: one read tells both that the words are
    // there and what they hold.  Bounded; if the words do not come the kernel waits for its
    // predecessors like kEarlyNone, and whatever it read is checked against the window kernel's
    // list after the wait, so no result depends on this phase.
    const int run = __ldcg(src.predictor_run);
    int ok = 0;
    for (int i = 0; i < kWatchPolls && !ok; ++i) ok = __syncthreads_and(read_words(run, true) ? 1 : 0);
    kEarly = ok ? kEarlyMask : kEarlyNone;
  } else if (kEarlyT == kEarlyMask) {
    read_words(0, false);                          // final before the kernel ahead passed its wait
  }
  if (kEarly == kEarlyNone) {
    pdl_wait();
    pdl_trigger();
  }
  int n;
  if (kEarly == kEarlyMask) {
    // block-wide prefix of the words' bit counts; the caller wants the want-th set bit
    int cnt = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) cnt += __popc(mw[i]);
    if (tid == 0) *first_id = -1;
    int off = block_exclusive_scan_256(cnt, &n, scan_sums);   // also orders the first_id store
    if (want >= off && want < off + cnt) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = __popc(mw[i]);
        if (want >= off && want < off + c) {
          uint32_t m = mw[i];
          for (int s = want - off; s > 0; --s) m &= m - 1;
          *first_id = (w0 + i) * src.word_bits + __ffs(m) - 1;
        }
        off += c;
      }
    }
    __syncthreads();
  } else {
    n = __ldcg(src.counts + LIF_CNT_N_LOAD);
  }
  EarlyPick pk;
  pk.mode = kEarly;
  pk.n = n;
  pk.id = kEarly == kEarlyMask ? *first_id : -1;
  return pk;
}


template <int kGate, int kEarlyT>
__global__ void __launch_bounds__(kThreads) fetch_ffn_kernel(FetchFfnArgs a) {
  __shared__ float part[kThreads / 32];
  __shared__ int scan_sums[kThreads / 32];
  __shared__ int first_id;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nvec = a.d >> 3;                       // 16-byte chunks per half row
  const EarlyPick pk = early_pick<kEarlyT>(a.early, blockIdx.x, scan_sums, &first_id);
  const int kEarly = pk.mode;
  int n = pk.n;
  uint4 up[kFusedChunks], down[kFusedChunks];
  auto host_loads = [&](int id) {
    const uint4* src = a.store + (size_t)id * 2 * nvec;
#pragma unroll
    for (int k = 0; k < kFusedChunks; ++k) {
      const int c = tid + k * kThreads;
      if (c < nvec) {
        up[k] = ld_stream16(src + c);
        down[k] = ld_stream16(src + nvec + c);
      }
    }
  };
  int j = blockIdx.x;
  int id = -1, slot = 0;
  const bool mine = j < n;                         // this CTA has a first bundle
  if (mine) {
    if (kEarly == kEarlyMask) {
      id = pk.id;
    } else {
      id = __ldcg(a.load_ids + j);
      slot = __ldcg(a.load_slots + j);
    }
    host_loads(id);
  }
  if (kEarly != kEarlyNone) {
    pdl_wait();
    pdl_trigger();
  }
  if (kEarly == kEarlyMask) {
    // The window kernel is complete.  Its list is the reference: the masks read ahead of the
    // wait are this step's exactly when count and id agree with it (they do not when the window
    // kernel refused the step — count 0, nothing is written — or when the masks were another
    // predictor run's); otherwise the CTA starts over from the list.
    const int n_plan = __ldcg(a.counts + LIF_CNT_N_LOAD);
    const bool stale = n_plan != n || (mine && __ldcg(a.load_ids + j) != id);
    n = n_plan;
    if (j < n) {
      slot = __ldcg(a.load_slots + j);
      if (stale) {
        id = __ldcg(a.load_ids + j);
        host_loads(id);
      }
    }
  }
  if (j >= n) return;                              // the sum reads min(grid, n) partials

  uint4 xq[kFusedChunks];
#pragma unroll
  for (int k = 0; k < kFusedChunks; ++k) {
    const int c = tid + k * kThreads;
    xq[k] = c < nvec ? reinterpret_cast<const uint4*>(a.x)[c] : make_uint4(0, 0, 0, 0);
  }
  float acc[kFusedChunks][8];
#pragma unroll
  for (int k = 0; k < kFusedChunks; ++k)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[k][e] = 0.f;

  while (true) {
    const float b = kGate == LIF_GATE_RESIDENT ? a.gate_val[id] : __half2float(a.bias[slot]);
    uint4* dst = a.cache + (size_t)slot * 2 * nvec;
    float p = 0.f;
#pragma unroll
    for (int k = 0; k < kFusedChunks; ++k) {
      const int c = tid + k * kThreads;
      if (c < nvec) {
        dst[c] = up[k];
        dst[nvec + c] = down[k];
        float uf[8], xf[8];
        unpack8(up[k], uf);
        unpack8(xq[k], xf);
#pragma unroll
        for (int e = 0; e < 8; ++e) p = fmaf(uf[e], xf[e], p);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
    if (lane == 0) part[warp] = p;
    __syncthreads();
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) v += part[w];
    const float h = kGate == LIF_GATE_RESIDENT ? apply_activation(b, a.act, a.act_thr) * v
                                               : apply_activation(v + b, a.act, a.act_thr);
    if (h != 0.f) {
#pragma unroll
      for (int k = 0; k < kFusedChunks; ++k) {
        if (tid + k * kThreads < nvec) {
          float df[8];
          unpack8(down[k], df);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[k][e] = fmaf(h, df[e], acc[k][e]);
        }
      }
    }
    j += gridDim.x;
    if (j >= n) break;
    __syncthreads();                               // part[] is free again
    id = a.load_ids[j];
    slot = a.load_slots[j];
    host_loads(id);
  }
  float4* out = reinterpret_cast<float4*>(a.y_partial + (size_t)blockIdx.x * a.d);
#pragma unroll
  for (int k = 0; k < kFusedChunks; ++k) {
    const int c = tid + k * kThreads;
    if (c < nvec) {
      out[2 * c] = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
      out[2 * c + 1] = make_float4(acc[k][4], acc[k][5], acc[k][6], acc[k][7]);
    }
  }
}

// The plain fetch with the same early start as fetch_ffn_kernel (used where that kernel does not
// apply: several input streams, three-vector bundles).  CTA c's first unit is slice c % slices
// of row c / slices of the load list; its host loads are issued ahead of the dependency wait
// and held in registers until the window kernel's list says where the row goes.  The units
// after the first come from the list.
template <int kEarlyT>
__global__ void __launch_bounds__(kThreads)
fetch_early_kernel(const uint4* __restrict__ store, uint4* __restrict__ cache,
                   const int32_t* __restrict__ load_ids, const int32_t* __restrict__ load_slots,
                   int row_vec, EarlySource early) {
  __shared__ int scan_sums[kThreads / 32];
  __shared__ int first_id;
  constexpr int kSlice = kThreads * kFetchUnroll;
  const int slices = (row_vec + kSlice - 1) / kSlice;
  const int j0 = blockIdx.x / slices;
  const int v0 = (blockIdx.x % slices) * kSlice + threadIdx.x;
  const EarlyPick pk = early_pick<kEarlyT>(early, j0, scan_sums, &first_id);
  uint4 buf[kFetchUnroll];
  auto host_loads = [&](int id) {
    const uint4* src = store + (size_t)id * row_vec;
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = v0 + i * kThreads;
      if (v < row_vec) buf[i] = ld_stream16(src + v);
    }
  };
  int n = pk.n, id = -1;
  const bool mine = j0 < n;
  if (mine) {
    id = pk.mode == kEarlyMask ? pk.id : __ldcg(load_ids + j0);
    host_loads(id);
  }
  if (pk.mode != kEarlyNone) {
    pdl_wait();
    pdl_trigger();
  }
  if (pk.mode == kEarlyMask) {
    // the window kernel's list is the reference (see fetch_ffn_kernel)
    const int n_plan = __ldcg(early.counts + LIF_CNT_N_LOAD);
    const bool stale = n_plan != n || (mine && __ldcg(load_ids + j0) != id);
    n = n_plan;
    if (j0 < n && stale) host_loads(__ldcg(load_ids + j0));
  }
  if (j0 < n) {
    uint4* dst = cache + (size_t)load_slots[j0] * row_vec;
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = v0 + i * kThreads;
      if (v < row_vec) dst[v] = buf[i];
    }
  }
  const long long units = (long long)n * slices;
  for (long long u = (long long)blockIdx.x + gridDim.x; u < units; u += gridDim.x) {
    const int j = (int)(u / slices);
    const int w0 = (int)(u % slices) * kSlice + threadIdx.x;
    const uint4* src = store + (size_t)load_ids[j] * row_vec;
    uint4* dst = cache + (size_t)load_slots[j] * row_vec;
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = w0 + i * kThreads;
      if (v < row_vec) buf[i] = ld_stream16(src + v);
    }
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const int v = w0 + i * kThreads;
      if (v < row_vec) dst[v] = buf[i];
    }
  }
}

__global__ void __launch_bounds__(kThreads)
probe_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n_chunks,
             int chunk_vec) {
  gather_rows(src, dst, nullptr, nullptr, n_chunks, chunk_vec);
}

// Streaming read of `n_vec` 16-byte vectors of device memory, eight loads in flight per thread,
// nothing else: the time such a launch takes is what any kernel that has to read that many bytes
// after its predecessor has finished can at best approach.  The xor of everything read goes to
// `sink` so that the loads cannot be dropped.
__global__ void __launch_bounds__(kThreads)
probe_read_kernel(const uint4* __restrict__ src, size_t n_vec, uint4* __restrict__ sink) {
  pdl_wait();
  pdl_trigger();
  uint4 acc = make_uint4(0, 0, 0, 0);
  const size_t stride = (size_t)gridDim.x * kThreads;
  size_t v = (size_t)blockIdx.x * kThreads + threadIdx.x;
  for (; v + 7 * stride < n_vec; v += 8 * stride) {
    uint4 q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = ld_stream16(src + v + i * stride);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      acc.x ^= q[i].x; acc.y ^= q[i].y; acc.z ^= q[i].z; acc.w ^= q[i].w;
    }
  }
  for (; v < n_vec; v += stride) {
    const uint4 q = ld_stream16(src + v);
    acc.x ^= q.x; acc.y ^= q.y; acc.z ^= q.z; acc.w ^= q.w;
  }
  if ((acc.x ^ acc.y ^ acc.z ^ acc.w) == 0x9e3779b9u) *sink = acc;   // practically never
}

// Streaming read through a shared-memory ring, the way the FFN kernels bring rows in: CTA c
// streams its share of `src` in pieces of `chunk` bytes through `stages` stages, refilled `group`
// stages at a time with one mbarrier per group (bounded waits); the only use of the data is one
// 4-byte read per thread and stage.  Stage s is filled by one bulk copy when mix_every == 0 or
// s % mix_every != 0, else by 16-byte asynchronous copies issued by all threads (cp.async, which
// goes through the load/store path instead of the bulk-copy engine).
__global__ void __launch_bounds__(kThreads)
probe_ring_kernel(const unsigned char* __restrict__ src, size_t bytes_per_cta, unsigned chunk,
                  int stages, int group, int mix_every, uint4* __restrict__ sink,
                  int32_t* __restrict__ timeouts) {
  extern __shared__ __align__(128) unsigned char ring[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + (size_t)stages * chunk);   // one per group
  const int tid = threadIdx.x;
  const unsigned char* mine = src + (size_t)blockIdx.x * bytes_per_cta;
  const int n_chunks = (int)(bytes_per_cta / chunk);
  const int n_groups = (n_chunks + group - 1) / group;
  const int ring_groups = stages / group;
  auto by_threads = [&](int s) { return mix_every > 0 && s % mix_every == 0; };
  if (tid == 0) {
    for (int g = 0; g < ring_groups; ++g) {
      int arrivals = 0;                       // per stage: one (bulk copy or skip) or one per thread
      for (int s = g * group; s < (g + 1) * group; ++s) arrivals += by_threads(s) ? kThreads : 1;
      mbar_init(bars + g, arrivals);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();
  __syncthreads();
  auto fill_group = [&](int g) {              // chunks of group g -> ring group g % ring_groups
    uint64_t* bar = bars + g % ring_groups;
    for (int j = 0; j < group; ++j) {
      const int c = g * group + j, s = (g % ring_groups) * group + j;
      const bool live = c < n_chunks;
      if (by_threads(s)) {
        if (live)
          for (unsigned off = (unsigned)tid * 16; off < chunk; off += kThreads * 16)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(ring + (size_t)s * chunk + off)),
                         "l"(mine + (size_t)c * chunk + off) : "memory");
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
      } else if (tid == j % kThreads) {
        if (live) {
          mbar_expect_tx(bar, chunk);
          bulk_g2s(ring + (size_t)s * chunk, mine + (size_t)c * chunk, chunk, bar);
        } else {
          mbar_arrive(bar);
        }
      }
    }
  };
  int issued = 0;                             // groups whose copies have been issued (uniform)
  for (; issued < min(ring_groups, n_groups); ++issued) fill_group(issued);
  unsigned acc = 0;
  for (int g = 0; g < n_groups; ++g) {
    const int lost = mbar_wait(bars + g % ring_groups, (unsigned)(g / ring_groups) & 1u) ? 0 : 1;
    for (int j = 0; j < group && g * group + j < n_chunks; ++j)
      acc ^= *reinterpret_cast<const unsigned*>(ring + (size_t)((g % ring_groups) * group + j) * chunk +
                                                (tid * 4) % chunk);
    if (__syncthreads_or(lost)) {             // give up: flag, let what is in flight land, leave
      if (tid == 0) atomicAdd(timeouts, 1);
      for (int gg = g + 1; gg < issued; ++gg)
        mbar_wait(bars + gg % ring_groups, (unsigned)(gg / ring_groups) & 1u);
      return;
    }
    // the generic-proxy reads of this group's stages are done: refill them
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (issued < n_groups) fill_group(issued++);
  }
  if (acc == 0x9e3779b9u) *sink = make_uint4(acc, 0, 0, 0);   // practically never
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

static EarlySource early_source(const lif_layer* L) {
  EarlySource e;
  e.entries = L->new_mask_words;
  e.nwords = new_mask_entries(L->desc);
  e.word_bits = new_mask_entry_bits(L->desc);
  e.predictor_run = L->counts + CNT_PREDICTOR_RUN;
  e.counts = L->counts;
  return e;
}

// The plain fetch behind the window kernel (or the row moves) on the same stream, started early
// (`early` as for launch_fetch_ffn).
cudaError_t launch_fetch_early(lif_layer* L, cudaStream_t st, int early) {
  if (early >= kEarlyMask && !fetch_ffn_can_watch(L)) early = kEarlyNone;
  if (early == kEarlyNone) return launch_fetch(L, st);
  auto kernel = early == kEarlyWatch  ? fetch_early_kernel<kEarlyWatch>
                : early == kEarlyMask ? fetch_early_kernel<kEarlyMask>
                                      : fetch_early_kernel<kEarlyLists>;
  return launch_k(kernel, dim3(L->fetch_grid), dim3(kThreads), 0, st, L->use_pdl,
                  (const uint4*)L->dev_bundles, (uint4*)L->desc.dev_cache,
                  (const int32_t*)L->load_ids, (const int32_t*)L->load_slots,
                  row_elems(L->desc) / 8, early_source(L));
}

// File-backed store: staging row j (bundle load_ids[j], read by the host) -> cache row load_slots[j].
cudaError_t launch_fetch_staged(lif_layer* L, cudaStream_t st) {
  return launch_k(fetch_kernel, dim3(L->fetch_grid), dim3(kThreads), 0, st, L->use_pdl,
                  (const uint4*)L->dev_bundles, (uint4*)L->desc.dev_cache, (const int32_t*)nullptr,
                  (const int32_t*)L->load_slots, (const int32_t*)L->counts, row_elems(L->desc) / 8);
}

bool fetch_ffn_supported(const lif_layer* L) {
  const lif_layer_desc& D = L->desc;
  return D.n_streams == 1 && D.gate_mode != LIF_GATE_BUNDLED &&
         D.d_model <= kFusedChunks * kThreads * 8 && L->fetch_grid == L->ffn_grid;
}

// The mask-driven forms scan at most four mask words per thread.
bool fetch_ffn_can_watch(const lif_layer* L) {
  return new_mask_entries(L->desc) <= 4 * kThreads;
}

// Fetch of this step's new rows fused with their FFN terms; partials go to `partial`
// ([fetch_grid][d_model], CTA c < min(grid, n_load) writes row c).
cudaError_t launch_fetch_ffn(lif_layer* L, const __half* x, float* partial, cudaStream_t st,
                             int early) {
  const lif_layer_desc& D = L->desc;
  FetchFfnArgs a;
  a.store = (const uint4*)L->dev_bundles;
  a.cache = (uint4*)D.dev_cache;
  a.load_ids = L->load_ids;
  a.load_slots = L->load_slots;
  a.counts = L->counts;
  a.bias = L->bias;
  a.x = x;
  a.gate_val = L->gate_val;
  a.y_partial = partial;
  a.d = D.d_model;
  a.act = D.activation;
  a.act_thr = D.activation_threshold;
  a.early = early_source(L);
  if (early >= kEarlyMask && !fetch_ffn_can_watch(L)) early = kEarlyNone;
  void (*kernel)(FetchFfnArgs);
  if (D.gate_mode == LIF_GATE_RESIDENT)
    kernel = early == kEarlyWatch   ? fetch_ffn_kernel<LIF_GATE_RESIDENT, kEarlyWatch>
             : early == kEarlyMask  ? fetch_ffn_kernel<LIF_GATE_RESIDENT, kEarlyMask>
             : early == kEarlyLists ? fetch_ffn_kernel<LIF_GATE_RESIDENT, kEarlyLists>
                                    : fetch_ffn_kernel<LIF_GATE_RESIDENT, kEarlyNone>;
  else
    kernel = early == kEarlyWatch   ? fetch_ffn_kernel<LIF_GATE_NONE, kEarlyWatch>
             : early == kEarlyMask  ? fetch_ffn_kernel<LIF_GATE_NONE, kEarlyMask>
             : early == kEarlyLists ? fetch_ffn_kernel<LIF_GATE_NONE, kEarlyLists>
                                    : fetch_ffn_kernel<LIF_GATE_NONE, kEarlyNone>;
  return launch_k(kernel, dim3(L->fetch_grid), dim3(kThreads), 0, st, L->use_pdl, a);
}

cudaError_t launch_probe_read(const void* dev_src, size_t bytes, void* dev_sink, int grid, int pdl,
                              cudaStream_t st) {
  return launch_k(probe_read_kernel, dim3(grid), dim3(kThreads), 0, st, pdl, (const uint4*)dev_src,
                  bytes / 16, (uint4*)dev_sink);
}

cudaError_t launch_probe_ring(const void* dev_src, size_t bytes_per_cta, unsigned chunk, int stages,
                              int group, int mix_every, int grid, void* dev_sink,
                              int32_t* dev_timeouts, cudaStream_t st) {
  const size_t smem = (size_t)stages * chunk + (size_t)(stages / group) * 8;
  cudaError_t e = cudaFuncSetAttribute(probe_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  return launch_k(probe_ring_kernel, dim3(grid), dim3(kThreads), smem, st, 1,
                  (const unsigned char*)dev_src, bytes_per_cta, chunk, stages, group, mix_every,
                  (uint4*)dev_sink, dev_timeouts);
}

cudaError_t launch_probe(const void* dev_src_alias, void* dev_dst, size_t bytes, size_t chunk,
                         int grid, cudaStream_t st) {
  probe_kernel<<<grid, kThreads, 0, st>>>((const uint4*)dev_src_alias, (uint4*)dev_dst,
                                          (int)(bytes / chunk), (int)(chunk / 16));
  return cudaGetLastError();
}

}  // namespace lif
