// Internal declarations shared by the translation units of liblif.so.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lif.h"
#include "lif_profile.h"

namespace lif {

// Private entries of the counts block (public ones: LIF_CNT_* in lif.h).
enum {
  CNT_TICKET_PREDICT = 16,  // "last block done" counter of the score kernel
  CNT_PREDICTOR_RUN = 17,   // number of the predictor run whose masks are (being) written
  CNT_TOTALS = 32           // four uint64: bytes_fetched, rows_moved, rows_active, rows_cached
};

constexpr int kNever = -(1 << 30);  // last_active stamp of a neuron never predicted active
constexpr int kThreads = 256;
constexpr int kWindowThreads = 1024;
// rows of A per CTA in the first predictor stage: about 32 CTAs, so stage 2 folds few partials
inline int z_rows_per_cta(int d_model) {
  const int rows = ((d_model + 31) / 32 + 31) / 32 * 32;
  return rows < 32 ? 32 : rows;
}
constexpr int kMaxZPartials = 32;   // z_cta_count() never exceeds it
inline int z_cta_count(int d_model) {
  return (d_model + z_rows_per_cta(d_model) - 1) / z_rows_per_cta(d_model);
}
constexpr int kLogitTile = 128;     // neurons per CTA in the second predictor stage
constexpr int kMaxStreams = 8;
constexpr int kTimingEvents = 10;   // z0 z1 s1 w1 m1 | f0 f1 | g0 g1 r1

struct Workspace {
  // offsets in bytes from the workspace base; every block 256-byte aligned
  size_t counts, pointers, slot_of, last_active, bias, active_idx, evict_ids, evict_slots,
      move_src, move_dst, load_ids, load_slots, active_slots, hit_slots, n_tmp, z_partial,
      mask_words, new_mask_words, keep_tok, h_rows, gate_val, y_partial, total;
};

// fp16 elements per bundle / cache row: up | down, preceded by the gate row when it is bundled
inline int row_elems(const lif_layer_desc& d) {
  return (d.gate_mode == LIF_GATE_BUNDLED ? 3 : 2) * d.d_model;
}

Workspace plan_workspace(const lif_layer_desc& d, int ffn_grid_max);

}  // namespace lif

struct lif_layer {
  lif_layer_desc desc;
  lif::Workspace ws;
  const __half* dev_bundles;  // device alias of desc.host_bundles
  int32_t* counts;
  int32_t *pointers, *slot_of, *last_active;
  __half* bias;
  int32_t *active_idx, *evict_ids, *evict_slots, *move_src, *move_dst, *load_ids, *load_slots,
      *active_slots, *hit_slots, *n_tmp;
  float* z_partial;
  uint32_t* mask_words;
  // Neurons predicted active that have no cache row yet, as 64-bit entries {bits, run}: the low
  // half holds the bits of 32 consecutive neurons (of one predictor CTA's neurons, where those
  // are fewer), the high half the number of the predictor run that stored it (one store).
  unsigned long long* new_mask_words;
  int8_t* keep_tok;   // [d_ff] last kept token per neuron (speculative mode)
  float* y_partial;
  float* h_rows;      // [K slices][d_ff][8] fp32: phase-A output of the multi-stream FFN
                      // (bundled gate: a second block of the same size for the up values)
  float* gate_val;    // [S][d_ff] fp32 gate pre-activations (resident gate only)
  // multi-stream (tensor-core) FFN configuration; fb_ok = 0: per-stream fallback
  int fb_ok, fb_up_stages, fb_parts, fb_cols, fb_partitions;
  int fb_ksplit, fb_kps, fb_up_partitions, fb_parts_min, fb_up_group, fb_up_two_ctas;
  size_t fb_up_smem, fb_down_smem;
  int n_sm;
  int z_ctas;         // CTAs of the first predictor stage
  int ffn_grid;       // CTAs of the sparse-FFN kernel
  int ffn_stages;     // bundles in flight per CTA
  int ffn_stages_max; // what fits the shared memory of one CTA
  size_t ffn_smem;    // dynamic shared memory of the sparse-FFN kernel
  int fetch_grid;     // CTAs of the fetch kernel
  int move_grid;
  unsigned wait_polls; // poll limit of the first wait on each bulk copy in the FFN kernels
  int early_fetch;    // knob: the plain fetch of lif_decode_step starts early behind the window kernel
  int watch_chain;    // set by lif_decode_step while it launches a step whose fetch kernel watches
                      // the predictor: window and row-move kernels release their dependents at entry
  int use_pdl;        // programmatic dependent launch along the compute stream
  int split_ffn;      // decode step: cached rows' FFN overlaps the fetch
  int fused_plan;     // decode step: window update reads the predictor's bit mask directly
  int fused_fetch;    // decode step: the fetch kernel also computes the new rows' FFN terms
  cudaEvent_t ev_plan, ev_fetch;
  // optional per-kernel timing: kTimingEvents events per recorded step
  cudaEvent_t* tm_events;
  int tm_steps, tm_cursor;
};

struct lif_graph {
  cudaGraph_t graph;
  cudaGraphExec_t exec;
  void* dev_x;
  float* dev_y;
  size_t x_bytes, y_bytes;
};

namespace lif {

// Timing events also work inside stream capture, where they become event-record nodes.
inline void tm_record(cudaEvent_t e, cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  cudaStreamIsCapturing(st, &cs);
  cudaEventRecordWithFlags(e, st, cs == cudaStreamCaptureStatusActive ? cudaEventRecordExternal
                                                                      : cudaEventRecordDefault);
}

// kernels' host launchers (each returns the launch's cudaError_t)
cudaError_t launch_reset(lif_layer* L, cudaStream_t st);
// `ev`: optional events of the current timed step (nullptr = no timing); each launcher
// records the ones between and after its own kernels.
cudaError_t launch_predict(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                           int32_t* n_active, cudaStream_t st, cudaEvent_t* ev = nullptr,
                           int compact = 1);   // compact = 0: leave only the bit mask
// Resident gate projection as the predictor: scores, threshold, bit mask, optional compaction.
cudaError_t launch_gate_predict(lif_layer* L, const __half* x, float* logits, int32_t* active_idx,
                                int32_t* n_active, cudaStream_t st, cudaEvent_t* ev, int compact);
bool window_plan_supported(const lif_layer_desc& D);
// with_moves = false: the caller launches the row moves itself (launch_moves)
cudaError_t launch_window_plan(lif_layer* L, cudaStream_t st, cudaEvent_t* ev = nullptr,
                               bool with_moves = true);
cudaError_t launch_window(lif_layer* L, const int32_t* act, const int32_t* n_act, cudaStream_t st,
                          cudaEvent_t* ev = nullptr, bool with_moves = true);
// release_early: the row-move kernel releases its dependent at entry (only ahead of a fetch
// kernel in its watching form)
cudaError_t launch_moves(lif_layer* L, cudaStream_t st, cudaEvent_t* ev = nullptr,
                         bool release_early = false);
cudaError_t launch_fetch(lif_layer* L, cudaStream_t st);
cudaError_t launch_fetch_staged(lif_layer* L, cudaStream_t st);
cudaError_t launch_fetch_early(lif_layer* L, cudaStream_t st, int early);
bool fetch_ffn_supported(const lif_layer* L);
bool fetch_ffn_can_watch(const lif_layer* L);
int gate_predict_tile();                           // neurons per CTA of the resident-gate predictor
// entries of new_mask_words and the neurons each one covers
inline int new_mask_entry_bits(const lif_layer_desc& D) {
  return D.gate_mode == LIF_GATE_RESIDENT ? gate_predict_tile() : 32;
}
inline int new_mask_entries(const lif_layer_desc& D) {
  if (D.gate_mode == LIF_GATE_RESIDENT) return (D.d_ff + gate_predict_tile() - 1) / gate_predict_tile();
  return (D.d_ff + kLogitTile - 1) / kLogitTile * (kLogitTile / 32);
}
// early: what the kernel may do before its own dependency wait.  kEarlyLists: the lists were
// final before the kernel ahead of this one passed its wait, so the first bundle's host loads
// are issued from them; kEarlyMask: the kernel ahead is the window kernel of the same step and
// the predictor ran just before that: the first bundle's id comes from the predictor's mask of
// neurons to bring in; kEarlyNone: nothing.
// kEarlyWatch: like kEarlyMask, but the window kernel ahead releases its dependents as soon as it
// starts, so this kernel is resident while the score kernel still runs and watches that kernel's
// count of finished tiles (bounded; it falls back to kEarlyNone when the count does not come).
enum { kEarlyNone = 0, kEarlyLists = 1, kEarlyMask = 2, kEarlyWatch = 3 };
cudaError_t launch_fetch_ffn(lif_layer* L, const __half* x, float* partial, cudaStream_t st,
                             int early);
cudaError_t launch_refill(lif_layer* L, cudaStream_t st);
cudaError_t launch_probe(const void* dev_src_alias, void* dev_dst, size_t bytes, size_t chunk,
                         int grid, cudaStream_t st);
cudaError_t launch_probe_read(const void* dev_src, size_t bytes, void* dev_sink, int grid, int pdl,
                              cudaStream_t st);
cudaError_t launch_probe_ring(const void* dev_src, size_t bytes_per_cta, unsigned chunk, int stages,
                              int group, int mix_every, int grid, void* dev_sink,
                              int32_t* dev_timeouts, cudaStream_t st);
// slots == nullptr: rows base[0] .. base[0] + n[0] (base == nullptr: 0)
cudaError_t launch_ffn(lif_layer* L, const __half* x, const int32_t* slots, const int32_t* n,
                       const int32_t* base, float* y, bool accumulate, cudaStream_t st,
                       cudaEvent_t* ev = nullptr);
cudaError_t launch_fetch_and_ffn_split(lif_layer* L, const __half* x, float* y, cudaStream_t st,
                                       cudaStream_t side, cudaEvent_t* ev = nullptr,
                                       bool moves_aside = false);
cudaError_t launch_one(lif_layer* L, int kernel, const __half* x, float* y, cudaStream_t st);
cudaError_t launch_predict_one(lif_layer* L, int kernel, const __half* x, cudaStream_t st);
cudaError_t ffn_configure(lif_layer* L);
constexpr int kBatchedMaxPartitions = 128;
constexpr int kBatchedMaxKSplit = 8;
// y[i] = b_down[i % d_model] + sum_{p < min(partitions, *n)} partial[p][i], i < width
cudaError_t launch_partial_sum(lif_layer* L, const float* partial, const int32_t* n,
                               int partitions, int width, float* y, cudaStream_t st);
bool ffn_batched_supported(const lif_layer_desc& D);
cudaError_t ffn_batched_configure(lif_layer* L);
cudaError_t launch_ffn_batched(lif_layer* L, const __half* x, const int32_t* slots,
                               const int32_t* n, const int32_t* base, float* y, cudaStream_t st);
size_t ffn_smem_for(const lif_layer* L, int stages);

// Launch with (pdl) or without the programmatic-stream-serialization attribute.  A kernel
// launched with it may start while the previous kernel of the stream is still running; it
// must execute pdl_wait() before it touches anything an earlier kernel wrote (every kernel of
// this library does so on every path, which also keeps the ordering transitive).  Inside a
// captured graph the attribute can make every incoming dependency of the launch programmatic,
// a cross-stream event wait included (measured: a kernel that read another stream's output
// ahead of its wait raced in graph replay only).  So what a kernel reads before pdl_wait() must
// be weights, or data that was final before each kernel ahead of it passed its own wait.
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                     cudaStream_t st, int pdl, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#ifdef __CUDACC__
// Block until every earlier kernel of the stream has completed and its writes are visible
// (no-op for a kernel launched without the attribute).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ float apply_activation(float v, int act, float thr) {
  if (act == LIF_ACT_RELU_SQUARED) {
    v = fmaxf(v, 0.f);
    return v * v;
  }
  if (act == LIF_ACT_FATRELU) return v > thr ? v : 0.f;
  return fmaxf(v, 0.f);
}
// Let the next kernel of the stream start its prologue.
__device__ __forceinline__ void pdl_trigger() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// 16-byte streaming load (no L1 allocation) of data that is read once: weights, bundles in
// mapped host memory.  Deliberately not the non-coherent (.nc) form: a load of memory the
// assembler knows to be read-only may be scheduled after a later griddepcontrol.wait, next to
// its first use, which silently turns a prefetch issued ahead of the dependency wait into a load
// behind it (measured: the predictor kernels 0.7-1 us slower each, the fetch kernel's early
// host loads without effect).  An ordinary load stays where it is written.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p)
               : "memory");
  return v;
}

// eight fp16 values -> fp32
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 t = __half22float2(h[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

// ---- mbarrier + bulk asynchronous copy (TMA, CTA-local, no multicast) -------------------------
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
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// Bounded wait: false if the phase did not complete within `limit` polls.
constexpr unsigned kWaitLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity,
                                          unsigned limit = kWaitLimit) {
  for (unsigned i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> this CTA's shared memory, completion counted in bytes on `bar`; src, dst and bytes
// are multiples of 16
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes,
                                         uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
#endif

}  // namespace lif
