// C ABI of liblif.so: argument checking, workspace carve-up and stream/event orchestration.
// Every step of the path runs in the kernels of predict.cu / window.cu / fetch.cu / ffn.cu.
#include <new>

#include "lif_internal.cuh"

namespace lif {

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

Workspace plan_workspace(const lif_layer_desc& d, int ffn_grid_max) {
  Workspace w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off = align_up(off + bytes, 256);
    return at;
  };
  const size_t F = d.d_ff, cap = d.capacity, S = d.n_streams;
  const size_t z_ctas = z_cta_count(d.d_model);
  const size_t n_mask = (F + kLogitTile - 1) / kLogitTile * (kLogitTile / 32);
  w.counts = take(LIF_CNT_LEN * 4);
  w.pointers = take(cap * 4);
  w.slot_of = take(F * 4);
  w.last_active = take(F * 4);
  w.bias = take(cap * 2);
  w.active_idx = take(F * 4);
  w.evict_ids = take(cap * 4);
  w.evict_slots = take(cap * 4);
  w.move_src = take(cap * 4);
  w.move_dst = take(cap * 4);
  w.load_ids = take(cap * 4);
  w.load_slots = take(cap * 4);
  w.active_slots = take(F * 4);
  w.hit_slots = take(F * 4);
  w.n_tmp = take(64);
  w.z_partial = take(z_ctas * S * d.rank * 4);
  w.mask_words = take(n_mask * 4);
  w.new_mask_words = take((size_t)new_mask_entries(d) * 8);
  w.keep_tok = take(d.spec_keep > 0 ? F : 0);
  w.h_rows = take(d.n_streams > 1 ? (size_t)kBatchedMaxKSplit * F * 8 * 4 *
                                        (d.gate_mode == LIF_GATE_BUNDLED ? 2 : 1)
                                  : 0);
  w.gate_val = take(d.gate_mode == LIF_GATE_RESIDENT ? S * F * 4 : 0);
  size_t partial_rows = (size_t)ffn_grid_max;
  if (ffn_batched_supported(d) && (size_t)kBatchedMaxPartitions * S > partial_rows)
    partial_rows = (size_t)kBatchedMaxPartitions * S;
  w.y_partial = take(partial_rows * d.d_model * 4);
  w.total = off;
  return w;
}

static int ffn_grid_upper_bound() { return 2 * 256; }   // >= 2 CTAs per SM on any part

static lif_status check_shape(const lif_layer_desc* d) {
  if (!d) return LIF_ERR_INVALID_ARG;
  if (d->d_model < 8 || d->d_model % 8 || d->d_model > 8192) return LIF_ERR_INVALID_ARG;
  if (d->d_ff < 8 || d->d_ff % 8 || d->d_ff >= (1 << 21)) return LIF_ERR_INVALID_ARG;
  if (d->rank < 8 || d->rank % 8 || d->rank > 2048) return LIF_ERR_INVALID_ARG;
  if (d->window_k < 1) return LIF_ERR_INVALID_ARG;
  if (d->capacity < 1 || d->capacity > d->d_ff) return LIF_ERR_INVALID_ARG;
  if (d->n_streams < 1 || d->n_streams > kMaxStreams) return LIF_ERR_INVALID_ARG;
  if (d->ffn_mode != 0 && d->ffn_mode != 1) return LIF_ERR_INVALID_ARG;
  if (d->budget_rows < 0 || d->budget_rows > d->capacity) return LIF_ERR_INVALID_ARG;
  if (d->spec_keep < 0 || d->spec_keep > d->n_streams) return LIF_ERR_INVALID_ARG;
  if (d->spec_keep > 0 && d->budget_rows > 0) return LIF_ERR_INVALID_ARG;
  if (d->budget_rows > 0 && d->window_k > 32) return LIF_ERR_INVALID_ARG;
  if (d->activation < LIF_ACT_RELU || d->activation > LIF_ACT_FATRELU) return LIF_ERR_INVALID_ARG;
  if (d->activation == LIF_ACT_FATRELU && !(d->activation_threshold >= 0.f)) return LIF_ERR_INVALID_ARG;
  if (!(d->threshold_logit == d->threshold_logit)) return LIF_ERR_INVALID_ARG;   // NaN
  if (d->gate_mode < LIF_GATE_NONE || d->gate_mode > LIF_GATE_RESIDENT) return LIF_ERR_INVALID_ARG;
  if (d->gate_mode == LIF_GATE_RESIDENT && d->spec_keep > 0) return LIF_ERR_INVALID_ARG;
  if (d->append_first != 0 && d->append_first != 1) return LIF_ERR_INVALID_ARG;
  if (d->append_first && d->ffn_mode == 1) return LIF_ERR_INVALID_ARG;
  if (d->staging_rows != 0 && (d->staging_rows < d->capacity || d->staging_rows > d->d_ff))
    return LIF_ERR_INVALID_ARG;
  return LIF_OK;
}

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

}  // namespace lif

using namespace lif;

extern "C" {

const char* lif_status_str(lif_status s) {
  switch (s) {
    case LIF_OK: return "ok";
    case LIF_ERR_INVALID_ARG: return "invalid argument";
    case LIF_ERR_ALIGNMENT: return "misaligned pointer";
    case LIF_ERR_CAPACITY: return "window cache capacity exceeded";
    case LIF_ERR_STATE: return "invalid state";
    case LIF_ERR_CUDA: return "CUDA error";
    case LIF_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown";
}

lif_status lif_workspace_bytes(const lif_layer_desc* desc, size_t* out_bytes) {
  if (!out_bytes) return LIF_ERR_INVALID_ARG;
  lif_status s = check_shape(desc);
  if (s != LIF_OK) return s;
  *out_bytes = plan_workspace(*desc, ffn_grid_upper_bound()).total;
  return LIF_OK;
}

lif_status lif_create_layer(const lif_layer_desc* desc, lif_layer** out) {
  if (!out) return LIF_ERR_INVALID_ARG;
  *out = nullptr;
  lif_status s = check_shape(desc);
  if (s != LIF_OK) return s;
  const bool resident = desc->gate_mode == LIF_GATE_RESIDENT;
  if (!desc->host_bundles || !desc->dev_bias_up || !desc->dev_cache || !desc->dev_workspace)
    return LIF_ERR_INVALID_ARG;
  if (resident ? !desc->dev_gate
               : (!desc->dev_pred_A || !desc->dev_pred_B || !desc->dev_pred_c))
    return LIF_ERR_INVALID_ARG;
  if (!aligned(desc->host_bundles, 16) || (resident && !aligned(desc->dev_gate, 16)) ||
      (!resident && (!aligned(desc->dev_pred_A, 16) || !aligned(desc->dev_pred_B, 16) ||
                     !aligned(desc->dev_pred_c, 4))) ||
      !aligned(desc->dev_bias_up, 2) || !aligned(desc->dev_cache, 16) ||
      !aligned(desc->dev_workspace, 256) ||
      (desc->dev_bias_down && !aligned(desc->dev_bias_down, 8)))
    return LIF_ERR_ALIGNMENT;
  Workspace ws = plan_workspace(*desc, ffn_grid_upper_bound());
  if (desc->workspace_bytes < ws.total) return LIF_ERR_INVALID_ARG;

  void* alias = nullptr;
  if (cudaHostGetDevicePointer(&alias, const_cast<void*>(desc->host_bundles), 0) != cudaSuccess) {
    cudaGetLastError();
    return LIF_ERR_INVALID_ARG;   // not pinned + mapped
  }
  lif_layer* L = new (std::nothrow) lif_layer();
  if (!L) return LIF_ERR_STATE;
  L->desc = *desc;
  L->ws = ws;
  L->dev_bundles = (const __half*)alias;
  unsigned char* b = (unsigned char*)desc->dev_workspace;
  L->counts = (int32_t*)(b + ws.counts);
  L->pointers = (int32_t*)(b + ws.pointers);
  L->slot_of = (int32_t*)(b + ws.slot_of);
  L->last_active = (int32_t*)(b + ws.last_active);
  L->bias = (__half*)(b + ws.bias);
  L->active_idx = (int32_t*)(b + ws.active_idx);
  L->evict_ids = (int32_t*)(b + ws.evict_ids);
  L->evict_slots = (int32_t*)(b + ws.evict_slots);
  L->move_src = (int32_t*)(b + ws.move_src);
  L->move_dst = (int32_t*)(b + ws.move_dst);
  L->load_ids = (int32_t*)(b + ws.load_ids);
  L->load_slots = (int32_t*)(b + ws.load_slots);
  L->active_slots = (int32_t*)(b + ws.active_slots);
  L->hit_slots = (int32_t*)(b + ws.hit_slots);
  L->n_tmp = (int32_t*)(b + ws.n_tmp);
  L->z_partial = (float*)(b + ws.z_partial);
  L->mask_words = (uint32_t*)(b + ws.mask_words);
  L->new_mask_words = (unsigned long long*)(b + ws.new_mask_words);
  L->keep_tok = desc->spec_keep > 0 ? (int8_t*)(b + ws.keep_tok) : nullptr;
  L->y_partial = (float*)(b + ws.y_partial);
  L->h_rows = (float*)(b + ws.h_rows);
  L->gate_val = resident ? (float*)(b + ws.gate_val) : nullptr;

  int dev = 0;
  bool ok = cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&L->n_sm, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess;
  ok = ok && ffn_configure(L) == cudaSuccess;
  L->fb_up_two_ctas = 0;
  L->early_fetch = 1;
  ok = ok && ffn_batched_configure(L) == cudaSuccess;
  if (ok) {
    L->z_ctas = z_cta_count(desc->d_model);
    L->ffn_grid = L->n_sm < ffn_grid_upper_bound() ? L->n_sm : ffn_grid_upper_bound();
    L->fetch_grid = L->n_sm;
    L->move_grid = L->n_sm;
    L->use_pdl = 1;
    L->wait_polls = kWaitLimit;
    L->split_ffn = 1;
    L->fused_plan = window_plan_supported(*desc) ? 1 : 0;
    L->fused_fetch = 1;
    ok = cudaEventCreateWithFlags(&L->ev_plan, cudaEventDisableTiming) == cudaSuccess;
    if (ok && cudaEventCreateWithFlags(&L->ev_fetch, cudaEventDisableTiming) != cudaSuccess) {
      cudaEventDestroy(L->ev_plan);
      ok = false;
    }
  }
  if (ok && launch_reset(L, 0) != cudaSuccess) {
    cudaEventDestroy(L->ev_plan);
    cudaEventDestroy(L->ev_fetch);
    ok = false;
  }
  if (!ok) {
    cudaGetLastError();
    delete L;
    return LIF_ERR_CUDA;
  }
  *out = L;
  return LIF_OK;
}

static void timing_free(lif_layer* L) {
  if (!L->tm_events) return;
  for (int i = 0; i < L->tm_steps * kTimingEvents; ++i) cudaEventDestroy(L->tm_events[i]);
  delete[] L->tm_events;
  L->tm_events = nullptr;
  L->tm_steps = L->tm_cursor = 0;
}

lif_status lif_timing_enable(lif_layer* L, int32_t n_steps) {
  if (!L || n_steps < 0 || n_steps > (1 << 20)) return LIF_ERR_INVALID_ARG;
  timing_free(L);
  if (n_steps == 0) return LIF_OK;
  const int n = n_steps * kTimingEvents;
  L->tm_events = new (std::nothrow) cudaEvent_t[n];
  if (!L->tm_events) return LIF_ERR_STATE;
  for (int i = 0; i < n; ++i) {
    if (cudaEventCreate(&L->tm_events[i]) != cudaSuccess) {
      for (int j = 0; j < i; ++j) cudaEventDestroy(L->tm_events[j]);
      delete[] L->tm_events;
      L->tm_events = nullptr;
      cudaGetLastError();
      return LIF_ERR_CUDA;
    }
  }
  L->tm_steps = n_steps;
  L->tm_cursor = 0;
  return LIF_OK;
}

lif_status lif_timing_read(lif_layer* L, float* us, int32_t* host_n_steps) {
  if (!L || !us || !host_n_steps) return LIF_ERR_INVALID_ARG;
  for (int p = 0; p < LIF_PHASE_LEN; ++p) us[p] = 0.f;
  *host_n_steps = 0;
  if (!L->tm_events) return LIF_ERR_STATE;
  if (cudaDeviceSynchronize() != cudaSuccess) return LIF_ERR_CUDA;
  // (first event, second event) of each phase within a step's event block
  static const int pairs[7][2] = {{0, 1}, {1, 2}, {2, 3}, {3, 4}, {5, 6}, {7, 8}, {8, 9}};
  for (int s = 0; s < L->tm_cursor; ++s) {
    cudaEvent_t* ev = L->tm_events + (size_t)s * kTimingEvents;
    for (int p = 0; p < 7; ++p) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ev[pairs[p][0]], ev[pairs[p][1]]) != cudaSuccess) {
        cudaGetLastError();
        return LIF_ERR_CUDA;
      }
      us[p] += ms * 1e3f;
    }
  }
  *host_n_steps = L->tm_cursor;
  return LIF_OK;
}

lif_status lif_destroy_layer(lif_layer* L) {
  if (!L) return LIF_ERR_INVALID_ARG;
  timing_free(L);
  cudaEventDestroy(L->ev_plan);
  cudaEventDestroy(L->ev_fetch);
  delete L;
  return LIF_OK;
}

lif_status lif_reset(lif_layer* L, void* stream) {
  if (!L) return LIF_ERR_INVALID_ARG;
  return launch_reset(L, (cudaStream_t)stream) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_predict(lif_layer* L, const void* dev_x, float* dev_logits_or_null,
                       int32_t* dev_active_idx, int32_t* dev_n_active, void* stream) {
  if (!L || !dev_x || !dev_active_idx || !dev_n_active) return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_x, 16) || !aligned(dev_active_idx, 4) || !aligned(dev_n_active, 4) ||
      (dev_logits_or_null && !aligned(dev_logits_or_null, 4)))
    return LIF_ERR_ALIGNMENT;
  return launch_predict(L, (const __half*)dev_x, dev_logits_or_null, dev_active_idx,
                        dev_n_active, (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_window_update(lif_layer* L, const int32_t* dev_active_idx,
                             const int32_t* dev_n_active, void* stream) {
  if (!L || !dev_active_idx || !dev_n_active) return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_active_idx, 4) || !aligned(dev_n_active, 4)) return LIF_ERR_ALIGNMENT;
  return launch_window(L, dev_active_idx, dev_n_active, (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_fetch_bundles(lif_layer* L, void* fetch_stream) {
  if (!L) return LIF_ERR_INVALID_ARG;
  if (L->desc.staging_rows) return LIF_ERR_STATE;     // host_bundles is not the store
  return launch_fetch(L, (cudaStream_t)fetch_stream) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_sparse_ffn(lif_layer* L, const void* dev_x, const int32_t* dev_slots,
                          const int32_t* dev_n_slots, float* dev_y, void* stream) {
  if (!L || !dev_x || !dev_n_slots || !dev_y) return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_x, 16) || !aligned(dev_y, 16) || !aligned(dev_n_slots, 4) ||
      (dev_slots && !aligned(dev_slots, 4)))
    return LIF_ERR_ALIGNMENT;
  return launch_ffn(L, (const __half*)dev_x, dev_slots, dev_n_slots, nullptr, dev_y, false,
                    (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_decode_step(lif_layer* L, const void* dev_x, float* dev_y, void* compute_stream,
                           void* fetch_stream) {
  if (!L || !dev_x || !dev_y) return LIF_ERR_INVALID_ARG;
  if (L->desc.staging_rows) return LIF_ERR_STATE;     // host_bundles is not the store
  if (!aligned(dev_x, 16) || !aligned(dev_y, 16)) return LIF_ERR_ALIGNMENT;
  cudaStream_t sc = (cudaStream_t)compute_stream, sf = (cudaStream_t)fetch_stream;
  const __half* x = (const __half*)dev_x;
  cudaEvent_t* ev = nullptr;
  if (L->tm_events && L->tm_cursor < L->tm_steps)
    ev = L->tm_events + (size_t)(L->tm_cursor++) * kTimingEvents;
  if (ev) tm_record(ev[0], sc);
  bool ok;
  // With append_first the row moves and the bundle writes touch different rows, so given a
  // second stream the moves leave the critical chain (they only precede the cached rows' FFN).
  const bool moves_aside = L->desc.append_first && sf != sc;
  // The fetch kernel can watch the predictor when it directly follows the window kernel (or the
  // row moves behind it) on the compute stream with dependent launches.  One input stream with
  // the FFN split around the fetch: two streams (the cached rows' FFN runs on the other).
  // Otherwise the plain fetch takes that place on the compute stream, and the second stream, if
  // there is one, carries the row moves.
  const bool split = L->split_ffn && L->desc.n_streams == 1;
  // (in speculative mode the load list is a subset of the predictor's mask: no early start)
  L->watch_chain = L->use_pdl && fetch_ffn_can_watch(L) && L->desc.spec_keep == 0 &&
                   (split ? sf != sc : L->early_fetch != 0);
  if (L->fused_plan) {
    ok = launch_predict(L, x, nullptr, L->active_idx, L->n_tmp, sc, ev, 0) == cudaSuccess;
    ok = ok && launch_window_plan(L, sc, ev, !moves_aside) == cudaSuccess;
  } else {
    ok = launch_predict(L, x, nullptr, L->active_idx, L->n_tmp, sc, ev) == cudaSuccess;
    ok = ok && launch_window(L, L->active_idx, L->n_tmp, sc, ev, !moves_aside) == cudaSuccess;
  }
  if (split) {
    ok = ok && launch_fetch_and_ffn_split(L, x, dev_y, sc, sf, ev, moves_aside) == cudaSuccess;
    L->watch_chain = 0;
    if (!ok) cudaGetLastError();
    return ok ? LIF_OK : LIF_ERR_CUDA;
  }
  if (L->watch_chain) {
    // compute stream: ... window kernel -> (row moves) -> fetch, resident early -> FFN
    L->watch_chain = 0;
    if (moves_aside) {                 // the moves touch other rows than the fetch: beside it
      ok = ok && cudaEventRecord(L->ev_plan, sc) == cudaSuccess;
      ok = ok && cudaStreamWaitEvent(sf, L->ev_plan, 0) == cudaSuccess;
      ok = ok && launch_moves(L, sf, ev) == cudaSuccess;
      ok = ok && cudaEventRecord(L->ev_fetch, sf) == cudaSuccess;
    }
    if (ev) tm_record(ev[5], sc);
    ok = ok && launch_fetch_early(L, sc, kEarlyWatch) == cudaSuccess;
    if (ev) tm_record(ev[6], sc);
    if (moves_aside) ok = ok && cudaStreamWaitEvent(sc, L->ev_fetch, 0) == cudaSuccess;
    if (L->desc.ffn_mode == 0)
      ok = ok && launch_ffn(L, x, L->active_slots, L->counts + LIF_CNT_N_ACTIVE, nullptr, dev_y,
                            false, sc, ev) == cudaSuccess;
    else
      ok = ok && launch_ffn(L, x, nullptr, L->counts + LIF_CNT_NUM_USED, nullptr, dev_y, false,
                            sc, ev) == cudaSuccess;
    if (!ok) cudaGetLastError();
    return ok ? LIF_OK : LIF_ERR_CUDA;
  }
  if (sf != sc) {
    ok = ok && cudaEventRecord(L->ev_plan, sc) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(sf, L->ev_plan, 0) == cudaSuccess;
  }
  if (moves_aside) ok = ok && launch_moves(L, sc, ev) == cudaSuccess;   // beside the fetch on sf
  if (ev) tm_record(ev[5], sf);
  ok = ok && launch_fetch(L, sf) == cudaSuccess;
  if (ev) tm_record(ev[6], sf);
  if (sf != sc) {
    ok = ok && cudaEventRecord(L->ev_fetch, sf) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(sc, L->ev_fetch, 0) == cudaSuccess;
  }
  if (L->desc.ffn_mode == 0)
    ok = ok && launch_ffn(L, x, L->active_slots, L->counts + LIF_CNT_N_ACTIVE, nullptr, dev_y,
                          false, sc, ev) == cudaSuccess;
  else
    ok = ok && launch_ffn(L, x, nullptr, L->counts + LIF_CNT_NUM_USED, nullptr, dev_y, false,
                          sc, ev) == cudaSuccess;
  if (!ok) cudaGetLastError();
  return ok ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_decode_token_host(lif_layer* const* layers, int32_t n_layers, const void* host_x,
                                 void* dev_x, float* dev_y, float* host_y, void* compute_stream,
                                 void* fetch_stream) {
  if (!layers || n_layers < 1 || !host_x || !dev_x || !dev_y || !host_y)
    return LIF_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l] || layers[l]->desc.d_model != layers[0]->desc.d_model ||
        layers[l]->desc.n_streams != layers[0]->desc.n_streams)
      return LIF_ERR_INVALID_ARG;
  cudaStream_t sc = (cudaStream_t)compute_stream;
  const size_t per = (size_t)layers[0]->desc.n_streams * layers[0]->desc.d_model;
  if (cudaMemcpyAsync(dev_x, host_x, per * 2, cudaMemcpyHostToDevice, sc) != cudaSuccess)
    return LIF_ERR_CUDA;
  for (int l = 0; l < n_layers; ++l) {
    lif_status s = lif_decode_step(layers[l], dev_x, dev_y + (size_t)l * per, compute_stream,
                                   fetch_stream);
    if (s != LIF_OK) return s;
  }
  if (cudaMemcpyAsync(host_y, dev_y, per * 4 * n_layers, cudaMemcpyDeviceToHost, sc) !=
      cudaSuccess)
    return LIF_ERR_CUDA;
  return cudaStreamSynchronize(sc) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_graph_capture(lif_layer* const* layers, int32_t n_layers, void* dev_x,
                             float* dev_y, void* compute_stream, void* fetch_stream,
                             lif_graph** out) {
  if (!out) return LIF_ERR_INVALID_ARG;
  *out = nullptr;
  if (!layers || n_layers < 1 || !dev_x || !dev_y || !compute_stream || !fetch_stream ||
      compute_stream == fetch_stream)
    return LIF_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l] || layers[l]->desc.d_model != layers[0]->desc.d_model ||
        layers[l]->desc.n_streams != layers[0]->desc.n_streams)
      return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_x, 16) || !aligned(dev_y, 16)) return LIF_ERR_ALIGNMENT;
  cudaStream_t sc = (cudaStream_t)compute_stream;
  const size_t per = (size_t)layers[0]->desc.n_streams * layers[0]->desc.d_model;
  lif_graph* g = new (std::nothrow) lif_graph();
  if (!g) return LIF_ERR_STATE;
  g->dev_x = dev_x;
  g->dev_y = dev_y;
  g->x_bytes = per * 2;
  g->y_bytes = per * 4 * n_layers;
  if (cudaStreamBeginCapture(sc, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    delete g;
    return LIF_ERR_CUDA;
  }
  lif_status s = LIF_OK;
  for (int l = 0; l < n_layers && s == LIF_OK; ++l)
    s = lif_decode_step(layers[l], dev_x, dev_y + (size_t)l * per, compute_stream, fetch_stream);
  cudaError_t e = cudaStreamEndCapture(sc, &g->graph);   // always end, also after an error
  if (s == LIF_OK && e == cudaSuccess && cudaGraphInstantiate(&g->exec, g->graph, 0) == cudaSuccess) {
    *out = g;
    return LIF_OK;
  }
  if (e == cudaSuccess && g->graph) cudaGraphDestroy(g->graph);
  cudaGetLastError();
  delete g;
  return s != LIF_OK ? s : LIF_ERR_CUDA;
}

lif_status lif_graph_launch(lif_graph* g, void* stream) {
  if (!g) return LIF_ERR_INVALID_ARG;
  return cudaGraphLaunch(g->exec, (cudaStream_t)stream) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_graph_launch_host(lif_graph* g, const void* host_x, float* host_y, void* stream) {
  if (!g || !host_x || !host_y) return LIF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  bool ok = cudaMemcpyAsync(g->dev_x, host_x, g->x_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  ok = ok && cudaGraphLaunch(g->exec, st) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(host_y, g->dev_y, g->y_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
  if (!ok) cudaGetLastError();
  return ok ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_graph_destroy(lif_graph* g) {
  if (!g) return LIF_ERR_INVALID_ARG;
  cudaGraphExecDestroy(g->exec);
  cudaGraphDestroy(g->graph);
  delete g;
  return LIF_OK;
}

lif_status lif_profile_launch(lif_layer* L, int32_t kernel, const void* dev_x, float* dev_y,
                              void* stream) {
  if (!L || !dev_x || L->desc.n_streams != 1) return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_x, 16) || (dev_y && !aligned(dev_y, 16))) return LIF_ERR_ALIGNMENT;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  switch (kernel) {
    case LIF_KERNEL_PREDICT_Z:     // only where the first stage is a kernel of its own
      if (L->desc.gate_mode == LIF_GATE_RESIDENT) return LIF_ERR_STATE;
      /* fall through */
    case LIF_KERNEL_PREDICT_SCORES:
      e = launch_predict_one(L, kernel, (const __half*)dev_x, st);
      break;
    case LIF_KERNEL_FETCH:     // in the form the decode step launches it
      if (L->desc.staging_rows) return LIF_ERR_STATE;
      e = (L->split_ffn && L->fused_fetch && fetch_ffn_supported(L))
              ? launch_fetch_ffn(L, (const __half*)dev_x,
                                 L->y_partial + (size_t)L->ffn_grid * L->desc.d_model, st,
                                 kEarlyLists)   // replayed on final lists
              : launch_fetch(L, st);
      break;
    case LIF_KERNEL_FFN_SUM:
      if (!dev_y) return LIF_ERR_INVALID_ARG;
      /* fall through */
    case LIF_KERNEL_FFN_ACTIVE:
    case LIF_KERNEL_FFN_HITS:
    case LIF_KERNEL_FFN_NEW:
    case LIF_KERNEL_FFN_CACHE:
      e = launch_one(L, kernel, (const __half*)dev_x, dev_y, st);
      break;
    default:
      return LIF_ERR_INVALID_ARG;
  }
  if (e != cudaSuccess) cudaGetLastError();
  return e == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_set_tuning(lif_layer* L, int32_t key, int32_t value) {
  if (!L) return LIF_ERR_INVALID_ARG;
  switch (key) {
    case LIF_TUNE_DEPENDENT_LAUNCH: L->use_pdl = value != 0; return LIF_OK;
    case LIF_TUNE_SPLIT_FFN: L->split_ffn = value != 0; return LIF_OK;
    case LIF_TUNE_FUSED_PLAN:
      L->fused_plan = value != 0 && window_plan_supported(L->desc);
      return LIF_OK;
    case LIF_TUNE_FUSED_FETCH_FFN: L->fused_fetch = value != 0; return LIF_OK;
    case LIF_TUNE_FETCH_CTAS:
      if (value < 1 || value > 4096) return LIF_ERR_INVALID_ARG;
      L->fetch_grid = value;
      return LIF_OK;
    case LIF_TUNE_FFN_CTAS:
      if (value < 1 || value > ffn_grid_upper_bound() / 2) return LIF_ERR_INVALID_ARG;
      L->ffn_grid = value;
      return LIF_OK;
    case LIF_TUNE_BATCHED_COLUMN_PARTS:
      if (value < 1 || value > 16) return LIF_ERR_INVALID_ARG;
      L->fb_parts_min = value;
      return ffn_batched_configure(L) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
    case LIF_TUNE_BATCHED_UP_TWO_CTAS:
      L->fb_up_two_ctas = value != 0;
      return ffn_batched_configure(L) == cudaSuccess ? LIF_OK : LIF_ERR_CUDA;
    case LIF_TUNE_EARLY_FETCH: L->early_fetch = value != 0; return LIF_OK;
    case LIF_TUNE_WAIT_POLLS:
      if (value < 0) return LIF_ERR_INVALID_ARG;
      L->wait_polls = (unsigned)value;
      return LIF_OK;
    case LIF_TUNE_FFN_STAGES:
      if (value < 1 || value > L->ffn_stages_max) return LIF_ERR_INVALID_ARG;
      L->ffn_stages = value;
      L->ffn_smem = ffn_smem_for(L, value);
      return LIF_OK;
  }
  return LIF_ERR_INVALID_ARG;
}

lif_status lif_get_lists(lif_layer* L, lif_lists* o) {
  if (!L || !o) return LIF_ERR_INVALID_ARG;
  o->counts = L->counts;
  o->active_idx = L->active_idx;
  o->evict_ids = L->evict_ids;
  o->move_src = L->move_src;
  o->move_dst = L->move_dst;
  o->load_ids = L->load_ids;
  o->load_slots = L->load_slots;
  o->active_slots = L->active_slots;
  o->hit_slots = L->hit_slots;
  o->pointers = L->pointers;
  o->slot_of = L->slot_of;
  o->last_active = L->last_active;
  o->bias = L->bias;
  o->keep_token = L->keep_tok;
  return LIF_OK;
}

// Window state that a snapshot holds, in this order: counts block, pointers, slot_of,
// last_active, bias.  The cache rows are not part of it: they are re-read from the host store.
namespace {
struct StatePart {
  void* dev;
  size_t bytes;
};
int state_parts(lif_layer* L, StatePart* p) {
  const size_t F = L->desc.d_ff, cap = L->desc.capacity;
  p[0] = {L->counts, LIF_CNT_LEN * 4};
  p[1] = {L->pointers, cap * 4};
  p[2] = {L->slot_of, F * 4};
  p[3] = {L->last_active, F * 4};
  p[4] = {L->bias, cap * 2};
  return 5;
}
}  // namespace

lif_status lif_read_state(lif_layer* L, int32_t* host_pointers, int32_t* host_slot_of,
                          int32_t* host_last_active, int32_t* host_num_used) {
  if (!L) return LIF_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return LIF_ERR_CUDA;
  const size_t F = L->desc.d_ff, cap = L->desc.capacity;
  bool ok = true;
  if (host_pointers)
    ok = ok && cudaMemcpy(host_pointers, L->pointers, cap * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (host_slot_of)
    ok = ok && cudaMemcpy(host_slot_of, L->slot_of, F * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (host_last_active)
    ok = ok && cudaMemcpy(host_last_active, L->last_active, F * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (host_num_used)
    ok = ok && cudaMemcpy(host_num_used, L->counts + LIF_CNT_NUM_USED, 4, cudaMemcpyDeviceToHost) ==
                   cudaSuccess;
  if (!ok) cudaGetLastError();
  return ok ? LIF_OK : LIF_ERR_CUDA;
}

lif_status lif_snapshot_bytes(lif_layer* L, size_t* out_bytes) {
  if (!L || !out_bytes) return LIF_ERR_INVALID_ARG;
  StatePart p[5];
  size_t total = 0;
  for (int i = 0, n = state_parts(L, p); i < n; ++i) total += p[i].bytes;
  *out_bytes = total;
  return LIF_OK;
}

lif_status lif_snapshot(lif_layer* L, void* host_buf, size_t bytes) {
  size_t need = 0;
  if (!L || !host_buf || lif_snapshot_bytes(L, &need) != LIF_OK || bytes < need)
    return LIF_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return LIF_ERR_CUDA;
  StatePart p[5];
  unsigned char* out = (unsigned char*)host_buf;
  for (int i = 0, n = state_parts(L, p); i < n; ++i) {
    if (cudaMemcpy(out, p[i].dev, p[i].bytes, cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return LIF_ERR_CUDA;
    }
    out += p[i].bytes;
  }
  return LIF_OK;
}

lif_status lif_restore(lif_layer* L, const void* host_buf, size_t bytes) {
  size_t need = 0;
  if (!L || !host_buf || lif_snapshot_bytes(L, &need) != LIF_OK || bytes < need)
    return LIF_ERR_INVALID_ARG;
  if (L->desc.staging_rows) return LIF_ERR_STATE;     // the rows cannot be re-read by neuron id
  // A snapshot of another shape, a truncated or a damaged one: everything the kernels will
  // use as an index is checked here, on the host, before any of it reaches the device.
  {
    const int F = L->desc.d_ff, cap = L->desc.capacity;
    const int32_t* cnt = (const int32_t*)host_buf;
    const int32_t* ptr = cnt + LIF_CNT_LEN;
    const int32_t* slot_of = ptr + cap;
    const int32_t* last = slot_of + F;
    const int n = cnt[LIF_CNT_NUM_USED], step = cnt[LIF_CNT_STEP];
    if (n < 0 || n > cap || step < 0) return LIF_ERR_STATE;
    for (int s = 0; s < cap; ++s) {
      if (s < n ? (ptr[s] < 0 || ptr[s] >= F || slot_of[ptr[s]] != s) : ptr[s] != -1)
        return LIF_ERR_STATE;
    }
    int cached = 0;
    for (int i = 0; i < F; ++i) {
      if (slot_of[i] >= 0) {
        if (slot_of[i] >= n || ptr[slot_of[i]] != i) return LIF_ERR_STATE;
        ++cached;
      } else if (slot_of[i] != -1) {
        return LIF_ERR_STATE;
      }
      if (last[i] >= step && last[i] != kNever) return LIF_ERR_STATE;   // stamps lie in the past
    }
    if (cached != n) return LIF_ERR_STATE;
  }
  if (cudaDeviceSynchronize() != cudaSuccess) return LIF_ERR_CUDA;
  StatePart p[5];
  const unsigned char* in = (const unsigned char*)host_buf;
  for (int i = 0, n = state_parts(L, p); i < n; ++i) {
    if (cudaMemcpy(p[i].dev, in, p[i].bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaGetLastError();
      return LIF_ERR_CUDA;
    }
    in += p[i].bytes;
  }
  if (launch_refill(L, 0) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    return LIF_ERR_CUDA;
  }
  return LIF_OK;
}

lif_status lif_get_stats(lif_layer* L, lif_stats* o) {
  if (!L || !o) return LIF_ERR_INVALID_ARG;
  int32_t host[LIF_CNT_LEN];
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(host, L->counts, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LIF_ERR_CUDA;
  }
  for (int i = 0; i < 16; ++i) o->counts[i] = host[i];
  const uint64_t* totals = reinterpret_cast<const uint64_t*>(host + CNT_TOTALS);
  o->bytes_fetched = totals[0];
  o->rows_moved = totals[1];
  o->rows_active = totals[2];
  o->rows_cached = totals[3];
  o->status = host[LIF_CNT_STATUS];
  o->reserved = 0;
  return LIF_OK;
}

lif_status lif_clear_status(lif_layer* L, void* stream) {
  if (!L) return LIF_ERR_INVALID_ARG;
  return cudaMemsetAsync(L->counts + LIF_CNT_STATUS, 0, 4, (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_probe_host_read(const void* host_src, void* dev_dst, size_t bytes,
                               size_t chunk_bytes, void* stream) {
  if (!host_src || !dev_dst || !bytes || !chunk_bytes) return LIF_ERR_INVALID_ARG;
  if (bytes % chunk_bytes || chunk_bytes % 16 || bytes / chunk_bytes > 0x7fffffff)
    return LIF_ERR_INVALID_ARG;
  if (!aligned(host_src, 16) || !aligned(dev_dst, 16)) return LIF_ERR_ALIGNMENT;
  void* alias = nullptr;
  if (cudaHostGetDevicePointer(&alias, const_cast<void*>(host_src), 0) != cudaSuccess) {
    cudaGetLastError();
    return LIF_ERR_INVALID_ARG;
  }
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return LIF_ERR_CUDA;
  return launch_probe(alias, dev_dst, bytes, chunk_bytes, n_sm, (cudaStream_t)stream) ==
                 cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_probe_device_read(const void* dev_src, size_t bytes, void* dev_sink,
                                 int32_t ctas_per_sm, int32_t dependent_launch, void* stream) {
  if (!dev_src || !dev_sink || !bytes || bytes % 16 || ctas_per_sm < 1 || ctas_per_sm > 8)
    return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_src, 16) || !aligned(dev_sink, 16)) return LIF_ERR_ALIGNMENT;
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return LIF_ERR_CUDA;
  return launch_probe_read(dev_src, bytes, dev_sink, n_sm * ctas_per_sm, dependent_launch != 0,
                           (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

lif_status lif_probe_bulk_ring(const void* dev_src, size_t bytes, uint32_t chunk_bytes,
                               int32_t stages, int32_t refill_group, int32_t ctas_per_sm,
                               int32_t threads_every, void* dev_sink, int32_t* dev_timeouts,
                               void* stream) {
  if (!dev_src || !dev_sink || !dev_timeouts || !bytes) return LIF_ERR_INVALID_ARG;
  if (chunk_bytes < 16 || chunk_bytes % 16 || stages < 1 || stages > 256 || refill_group < 1 ||
      refill_group > stages || stages % refill_group || ctas_per_sm < 1 || ctas_per_sm > 8 ||
      threads_every < 0)
    return LIF_ERR_INVALID_ARG;
  if (!aligned(dev_src, 16) || !aligned(dev_sink, 16) || !aligned(dev_timeouts, 4))
    return LIF_ERR_ALIGNMENT;
  int dev = 0, n_sm = 0, max_smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
    return LIF_ERR_CUDA;
  if ((size_t)stages * chunk_bytes + (size_t)stages * 8 > (size_t)max_smem) return LIF_ERR_INVALID_ARG;
  const int grid = n_sm * ctas_per_sm;
  const size_t per_cta = bytes / grid / chunk_bytes * chunk_bytes;   // whole chunks, 16-byte aligned
  if (per_cta == 0) return LIF_ERR_INVALID_ARG;
  return launch_probe_ring(dev_src, per_cta, chunk_bytes, stages, refill_group, threads_every, grid,
                           dev_sink, dev_timeouts, (cudaStream_t)stream) == cudaSuccess
             ? LIF_OK
             : LIF_ERR_CUDA;
}

}  // extern "C"
