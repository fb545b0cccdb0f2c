/*
 * lif.h — C ABI of the sparse-decode FFN path of "LLM in a flash" (arXiv 2312.11514),
 * implemented as CUDA kernels for sm_100a.
 *
 * One `lif_layer` is one FFN layer of a ReLU transformer whose full weights live in a
 * row-column-bundle store in pinned host memory (standing in for flash) and whose recently
 * used neurons live in a preallocated cache in device memory (Section 3.3: `matrix`,
 * `pointers`, `bias`, `num_used`, `last_k_active`).
 *
 * Conventions
 *  - "dev" pointers are device addresses, "host" pointers are host addresses.  The caller
 *    owns every buffer it passes and keeps it alive until lif_destroy_layer; the library owns
 *    only the opaque handle (plus two CUDA events inside it).
 *  - `stream` arguments are `cudaStream_t` values passed as `void*` (NULL = default stream).
 *  - Calls that take a stream only enqueue work and never synchronise.  Argument errors are
 *    returned immediately.  Conditions only the device can see are written to the layer's
 *    sticky device status word and reported by lif_get_stats: a cache overflow or a bad neuron
 *    id (the window update of that step is refused, the window state untouched); a row index
 *    outside the cache given to the sparse FFN (the row is not read and contributes nothing); a
 *    bounded wait on a copy that ran out (LIF_ERR_TIMEOUT: that call's output lacks some rows'
 *    terms; the window bookkeeping stays consistent, and while this status stands every
 *    further window update is refused — lif_clear_status resumes).
 *  - fp16 = IEEE binary16; accumulations are fp32.
 *  - All counts the kernels need (n_active, n_load, ...) stay in device memory; no call
 *    needs them on the host to launch the next one.
 */
#ifndef LIF_H
#define LIF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LIF_OK = 0,
  LIF_ERR_INVALID_ARG = 1,
  LIF_ERR_ALIGNMENT = 2,
  LIF_ERR_CAPACITY = 3, /* window union would exceed `capacity` rows */
  LIF_ERR_STATE = 4,
  LIF_ERR_CUDA = 5,
  LIF_ERR_TIMEOUT = 6   /* a bounded device-side wait gave up */
} lif_status;

const char* lif_status_str(lif_status s);

/* FFN non-linearities the paper runs (Appendix C): ReLU for OPT and the relufied Falcon and
 * Phi-2; squared ReLU for Persimmon 8B; FATReLU for the sparsified Llama 2 — a neuron passes
 * its pre-activation v only when v > activation_threshold (threshold 0 is ReLU). */
enum { LIF_ACT_RELU = 0, LIF_ACT_RELU_SQUARED = 1, LIF_ACT_FATRELU = 2 };

/* Gated FFN (Appendix C, Llama 2: a gated linear unit, an up and a down projection; the
 * activation is applied to the gate value):
 *   y = b_down + sum_i act(<gate_i, x> + bias_i) * <up_i, x> * down_i.
 * LIF_GATE_NONE      plain FFN, bundle = up row | down column (Section 3.2).
 * LIF_GATE_BUNDLED   the gate row travels with the neuron: bundle and cache row are
 *                    gate | up | down, 6*d_model bytes; the low-rank predictor decides what to
 *                    load; bias_up is the gate's bias.
 * LIF_GATE_RESIDENT  the gate projection stays in device memory and is the predictor
 *                    (Appendix C, Llama 2, "alternative approaches"): score_i = <gate_i, x> +
 *                    bias_i exactly, a neuron is active iff its score exceeds the activation's
 *                    threshold (activation_threshold for FATReLU, 0 otherwise) for at least one
 *                    stream, bundles are up | down, and the FFN reuses the scores as gate
 *                    values.  dev_pred_A/B/c, rank and threshold_logit are ignored. */
enum { LIF_GATE_NONE = 0, LIF_GATE_BUNDLED = 1, LIF_GATE_RESIDENT = 2 };

typedef struct lif_layer lif_layer;

/* Layer description.  Shapes follow Section 3.3: the cache `matrix` is
 * [capacity][V*d_model]; row s holds up-projection row `pointers[s]` followed by
 * down-projection column `pointers[s]` (Section 3.2, bundling columns and rows), preceded by
 * the gate row when gate_mode is LIF_GATE_BUNDLED.  V = 3 in that mode, 2 otherwise. */
typedef struct {
  int32_t d_model;          /* multiple of 8, <= 8192 */
  int32_t d_ff;             /* multiple of 8, < 2^21 */
  int32_t rank;             /* predictor rank r, multiple of 8, <= 2048 */
  int32_t window_k;         /* tokens kept in the window, current one included, >= 1 */
  int32_t capacity;         /* rows of the cache (the paper's Req_i), 1..d_ff */
  int32_t n_streams;        /* S: concurrent decode streams sharing the layer, 1..8 */
  float threshold_logit;    /* theta: neuron active iff score > theta; sigmoid threshold tau
                               maps to ln(tau/(1-tau)), tau = 0.5 -> 0 (Section 3.1, App. B) */
  int32_t ffn_mode;         /* 0: FFN over the rows of the currently active neurons;
                               1: over every cached row [0, num_used) (Section 3.3 item 3) */
  int32_t activation;       /* LIF_ACT_*: the FFN non-linearity applied to <up row, x> + bias */
  float activation_threshold; /* FATReLU threshold (LIF_ACT_FATRELU only; >= 0) */
  int32_t budget_rows;      /* 0 = off.  Memory budget (Appendix C, Persimmon 8B / Phi-2): rows
                               the cache may hold, <= capacity.  When a step would pass it, that
                               step deletes with the widest window k' <= window_k (at least 1)
                               that fits; LIF_CNT_K_EFF reports k'.  Needs window_k <= 32. */
  int32_t spec_keep;        /* 0 = off.  Speculative decoding (Section 4): the n_streams inputs of
                               a step are consecutive tokens of one sequence and the window is
                               updated with all of them at once, keeping the last window_k
                               tokens that end with token spec_keep (1..n_streams) of the
                               step; a neuron active only in later tokens is used by this
                               step but gets the oldest stamp still inside the window.  The
                               step counter advances by spec_keep.  Not with budget_rows. */
  int32_t gate_mode;        /* LIF_GATE_*.  LIF_GATE_RESIDENT: not with spec_keep */
  int32_t append_first;     /* 0: the order of Section 3.3 — delete (last rows move into the freed
                               ones), then stack the new neurons at the end.  1: stack first,
                               then delete: the last rows are then new neurons, so their bundles
                               are written straight into freed rows and only deletions that
                               outnumber the arrivals move cached rows.  Same cached set and
                               outputs, fewer row copies, and row moves no longer touch the
                               rows the fetch writes.  Not with ffn_mode = 1. */
  int32_t staging_rows;     /* 0: host_bundles is the whole bundle store.  > 0 (>= capacity): the
                               bundles live in a file (lif_store_*) and host_bundles is only a
                               staging buffer of this many rows; the layer then steps through
                               lif_decode_step_store, and the calls that read the store by
                               neuron id (lif_fetch_bundles, lif_decode_step, graphs, lif_restore)
                               return LIF_ERR_STATE */
  const void* dev_gate;     /* LIF_GATE_RESIDENT: fp16 [d_ff][d_model] gate projection, 16-byte
                               aligned; otherwise ignored */
  const void* host_bundles; /* HOST, pinned + mapped: fp16 [d_ff][V*d_model]
                               (staging_rows > 0: [staging_rows][V*d_model]) */
  const void* dev_pred_A;   /* fp16 [d_model][rank] */
  const void* dev_pred_B;   /* fp16 [rank][d_ff] */
  const float* dev_pred_c;  /* fp32 [d_ff] per-neuron score offset */
  const void* dev_bias_up;  /* fp16 [d_ff]: up-projection (gated: gate) biases, always resident */
  const void* dev_bias_down;/* fp16 [d_model] or NULL */
  void* dev_cache;          /* fp16 [capacity][V*d_model], 16-byte aligned */
  void* dev_workspace;      /* 256-byte aligned, lif_workspace_bytes() bytes; holds the window
                               state and all lists; initialised by lif_create_layer's reset */
  size_t workspace_bytes;
} lif_layer_desc;

/* Indices into the device counts block (int32[LIF_CNT_LEN]). */
enum {
  LIF_CNT_N_ACTIVE = 0,     /* neurons predicted active this step */
  LIF_CNT_N_EVICT = 1,      /* neurons that left the window */
  LIF_CNT_N_MOVES = 2,      /* rows moved from the tail into freed slots */
  LIF_CNT_N_LOAD = 3,       /* neurons to bring in */
  LIF_CNT_N_HITS = 4,       /* active neurons already cached */
  LIF_CNT_NUM_USED_BEFORE = 5,
  LIF_CNT_NUM_KEPT = 6,     /* rows left after deleting (without append_first also the first
                               row of the new neurons) */
  LIF_CNT_NUM_USED = 7,     /* rows in use after the step */
  LIF_CNT_STEP = 8,         /* steps applied so far */
  LIF_CNT_STATUS = 9,       /* sticky lif_status written by kernels */
  LIF_CNT_K_EFF = 10,       /* window actually applied this step (= window_k without a budget) */
  LIF_CNT_LEN = 64
};

/* Device addresses of the per-step lists and of the window state, all inside the
 * workspace.  Lists are int32 and valid after lif_window_update of the same step:
 *   active_idx[n_active]   ascending neuron ids (as given to lif_window_update)
 *   evict_ids[n_evict]     deleted neurons in ascending order of the slot they held
 *   move_src/dst[n_moves]  row move_src[j] was copied to row move_dst[j]
 *   load_ids[n_load]       neurons to bring in, ascending id; load_slots[j] = num_kept + j
 *                          (append_first: the freed rows first, see lif_layer_desc)
 *   active_slots[n_active] cache row of active_idx[q] after the update
 *   hit_slots[n_hits]      rows of the active neurons that were already cached
 * State: pointers[capacity] (row -> neuron, -1 = free), slot_of[d_ff] (neuron -> row, -1 =
 * absent), last_active[d_ff] (last step predicted active), bias[capacity] fp16. */
typedef struct {
  int32_t* counts;
  int32_t* active_idx;
  int32_t* evict_ids;
  int32_t* move_src;
  int32_t* move_dst;
  int32_t* load_ids;
  int32_t* load_slots;
  int32_t* active_slots;
  int32_t* hit_slots;
  int32_t* pointers;
  int32_t* slot_of;
  int32_t* last_active;
  void* bias;
  int8_t* keep_token;       /* [d_ff], spec_keep > 0 only: per neuron, the last token j <
                               spec_keep of the step in which it is active, -1 if none; written
                               by lif_predict, read by lif_window_update for the active ones */
} lif_lists;

typedef struct {
  int32_t counts[16];       /* counts block entries 0..15 of the last step */
  uint64_t bytes_fetched;   /* cumulative: sum of n_load * bundle bytes */
  uint64_t rows_moved;      /* cumulative */
  uint64_t rows_active;     /* cumulative: sum of n_active over steps */
  uint64_t rows_cached;     /* cumulative: sum of num_used over steps */
  int32_t status;           /* sticky device status (lif_status) */
  int32_t reserved;
} lif_stats;

/* Bytes of device workspace a layer of this description needs (pointer fields ignored). */
lif_status lif_workspace_bytes(const lif_layer_desc* desc, size_t* out_bytes);

/* Validate `desc` (sizes, NULLs, 16-byte alignment, host_bundles registered as mapped pinned
 * memory), create the handle and enqueue a cold-cache reset on the default stream.
 * Allocates no device memory.  Section 3.3: num_used starts at zero. */
lif_status lif_create_layer(const lif_layer_desc* desc, lif_layer** out);

/* Frees the handle and its events; never touches caller memory. */
lif_status lif_destroy_layer(lif_layer* layer);

/* Empty the cache and restart the step counter (cold start). */
lif_status lif_reset(lif_layer* layer, void* stream);

/* Low-rank predictor (Section 3.1, "Anticipating ReLU Sparsity"): scores = x.A.B + c in fp32,
 * active iff score > theta for at least one stream.  With LIF_GATE_RESIDENT the scores are the
 * gate pre-activations <gate_i, x> + bias_i and theta is the activation's threshold.
 *   dev_x              fp16 [n_streams][d_model]
 *   dev_logits_or_null fp32 [n_streams][d_ff] scores (optional)
 *   dev_active_idx     int32 [d_ff]: ascending ids of the active neurons
 *   dev_n_active       int32 [1] */
lif_status lif_predict(lif_layer* layer, const void* dev_x, float* dev_logits_or_null,
                       int32_t* dev_active_idx, int32_t* dev_n_active, void* stream);

/* Sliding-window update (Section 3.1 "The Sliding Window Technique", Section 3.3 items 1-2):
 * stamps the active neurons, deletes the neurons not active in the last window_k steps by
 * moving tail rows into their slots (first freed slot <- last surviving row), assigns rows
 * num_kept.. (append_first: freed rows first) to the neurons to bring in (ascending id),
 * updates pointers / slot_of / bias / num_used, writes every list of lif_lists, applies the row moves inside dev_cache, and
 * advances the step.  On overflow sets LIF_ERR_CAPACITY in the status word and changes
 * nothing.  dev_active_idx must be ascending and duplicate-free. */
lif_status lif_window_update(lif_layer* layer, const int32_t* dev_active_idx,
                             const int32_t* dev_n_active, void* stream);

/* Bring in new neurons (Section 3.3 item 2): copy bundle load_ids[j] from the host store to
 * cache row load_slots[j], reading host memory directly from the kernel. */
lif_status lif_fetch_bundles(lif_layer* layer, void* fetch_stream);

/* Inference over cached rows (Section 3.3 item 3):
 *   y[s] = b_down + sum_q act(<matrix[slot_q, :d], x[s]> + bias[slot_q]) * matrix[slot_q, d:]
 * (gated layers: see LIF_GATE_*; with LIF_GATE_RESIDENT the gate values are those of the last
 * lif_predict / lif_decode_step of the layer, which must have been given the same x)
 *   dev_slots    int32 rows to use, or NULL for rows [0, *dev_n_slots)
 *   dev_n_slots  int32 [1] (device)
 *   dev_y        fp32 [n_streams][d_model]
 * A row outside [0, capacity) or a count outside [0, capacity] is never used to address the
 * cache: the row contributes nothing, the count is clamped, and the status word becomes
 * LIF_ERR_INVALID_ARG. */
lif_status lif_sparse_ffn(lif_layer* layer, const void* dev_x, const int32_t* dev_slots,
                          const int32_t* dev_n_slots, float* dev_y, void* stream);

/* Sparse FFN for callers that cannot allocate device memory.  (The paper has no counterpart
 * to this call; it exists for integration.)  lif_sparse_ffn needs a layer, and a layer needs
 * a caller-allocated workspace for the per-CTA partial sums.  Code that runs where allocation
 * is off limits — inside another framework's plugin or callback that owns the allocator, in a
 * process whose device memory was fully handed out at start-up, or in a code path that must
 * not synchronise the device, which cudaMalloc and cudaFree may do — can call this variant
 * instead: the partial sums live in a fixed 2 MiB array inside the library's device image
 * (held on every GPU that loads the library until the process exits), and the call allocates
 * nothing, on the host or the device.
 *   dev_matrix     fp16 [n_rows][2*d_model] cache rows (up half, down half), 16-byte aligned
 *   n_rows         rows of dev_matrix (>= 1): a row index outside [0, n_rows), or a count
 *                  outside [0, n_rows], is never used to address memory; it contributes
 *                  nothing (the count is clamped) and is reported as LIF_ERR_INVALID_ARG by
 *                  lif_sparse_ffn_static_status
 *   dev_bias       fp16 [n_rows] up-projection bias of each row
 *   dev_x          fp16 [d_model], one stream
 *   dev_slots      int32 rows to use, or NULL for rows [0, *dev_n_slots)
 *   dev_n_slots    int32 [1] on the device
 *   dev_bias_down  fp16 [d_model] or NULL
 *   dev_y          fp32 [d_model]
 * Same arithmetic as lif_sparse_ffn, but the number of CTAs (at most 2 MiB / (4*d_model) and
 * at most one per SM) and therefore the order of the partial sums can differ, so results
 * agree to rounding, not bitwise.  d_model above LIF_STATIC_MAX_D_MODEL, or not a multiple of
 * 8, is refused with LIF_ERR_INVALID_ARG; misaligned pointers with LIF_ERR_ALIGNMENT.
 * The first call on each device (of either function below) looks up the array's device
 * address and opts the kernel in to large shared memory; make that first call with the device
 * current and outside any stream capture.  All calls on a device share the one array and it
 * keeps the previous call's contents: every call overwrites the part it reads, but two calls
 * whose kernels overlap on the GPU (different streams) race on it — keep calls on one device
 * ordered.
 * Conditions only the kernels can see go to a status word inside the same array, which stays
 * set until it is read: lif_sparse_ffn_static_status synchronises the device, copies the word
 * (a lif_status: LIF_OK, LIF_ERR_INVALID_ARG for a refused row or count, LIF_ERR_TIMEOUT for a
 * bounded wait that ran out — the output of that call then lacks some rows' terms) to
 * *host_status and, with clear != 0, resets it.  It allocates nothing either. */
#define LIF_STATIC_MAX_D_MODEL 8192
lif_status lif_sparse_ffn_static(const void* dev_matrix, int32_t n_rows, const void* dev_bias,
                                 const void* dev_x, const int32_t* dev_slots,
                                 const int32_t* dev_n_slots, const void* dev_bias_down,
                                 float* dev_y, int32_t d_model, void* stream);
lif_status lif_sparse_ffn_static_status(int32_t* host_status, int32_t clear);

/* The bundle store in a file: the paper's storage tier.  Section 2.2 ("Read Throughput"),
 * Section 4.1 ("Implementation Details") and Appendix C ("Caching Considerations for Data Loading
 * from Flash Memory"): the bundles of the newly needed neurons are read from flash by many
 * threads (32 in the paper), one read per bundle, bypassing the operating system's cache, and
 * the loads are managed on the CPU.
 * lif_store_open: `path` holds n_bundles bundles of bundle_bytes bytes each (multiple of 16),
 * bundle i at byte i * bundle_bytes; n_threads reader threads (1..256) are started.  direct_io != 0
 * asks for uncached reads (O_DIRECT); where the file system refuses, the file is read through the
 * cache and lif_store_stats.direct_io says so.  Bundles whose size or destination is not a
 * multiple of 4096 bytes are read through an aligned window and copied.
 * lif_store_read: bundles host_ids[0..n) into host_dst[j * bundle_bytes], with the store's
 * threads; returns when all are read.  LIF_ERR_INVALID_ARG for an id outside the store,
 * LIF_ERR_STATE for a failed read.  One call at a time per store.
 * lif_decode_step_store: one token through a layer created with staging_rows > 0 — predict and
 * window update on the device, the load list copied to the host (the stream is synchronised),
 * the bundles read from the file into the staging buffer, copied to their cache rows by a kernel,
 * and the sparse FFN; the stream is synchronised again before the call returns (the staging
 * buffer is free for the next step).  Same results as lif_decode_step on a pinned store. */
typedef struct lif_store lif_store;
typedef struct {
  uint64_t reads;           /* read calls issued */
  uint64_t bytes_read;      /* bytes those calls returned (aligned windows included) */
  uint64_t bytes_requested; /* bundles asked for x bundle_bytes */
  double seconds_reading;   /* wall time inside batches of reads */
  int32_t direct_io;        /* 1: the file is open for uncached reads */
  int32_t n_threads;
} lif_store_stats;
lif_status lif_store_open(const char* path, int64_t n_bundles, int64_t bundle_bytes,
                          int32_t n_threads, int32_t direct_io, lif_store** out);
lif_status lif_store_close(lif_store* store);
lif_status lif_store_read(lif_store* store, const int32_t* host_ids, int32_t n, void* host_dst);
lif_status lif_store_get_stats(lif_store* store, lif_store_stats* host_out);
lif_status lif_decode_step_store(lif_layer* layer, lif_store* store, const void* dev_x, float* dev_y,
                                 void* stream);

/* Neuron sharding over several devices (not in the paper, which runs on one device; it rests
 * on Section 3.3 item 3: the FFN output is a sum of one term per cached neuron, in any order).
 * Each device creates its layers over its own share of the neurons (its rows of the bundle
 * store, its columns of dev_pred_B, its entries of dev_pred_c and dev_bias_up; dev_bias_down on
 * one device only), runs the calls above on them, and the layer's output is the sum over devices
 * of the outputs computed there.
 * lif_sum_peer_outputs forms that sum on the calling device:
 *   dev_y[i] = dev_partials[0][i] + dev_partials[1][i] + ... (in this order), i < n_floats.
 *   dev_partials  HOST array of n_peers device pointers, fp32, 16-byte aligned; each is the
 *                 partial output of one device ([n_streams][d_model] of one layer, or several
 *                 layers' worth): memory of the current device, or of a peer device that is
 *                 mapped into this one (peer access enabled, or a shared mapping).  Read with
 *                 plain loads.  The array itself is read during the call only.
 *   n_peers       1 .. LIF_MAX_PEERS
 *   dev_y         fp32 [n_floats] on the current device, 16-byte aligned; may be exactly one of
 *                 the partials (the sum then replaces it), but not a shifted overlap of one.
 *   n_floats      multiple of 4
 * Enqueue only.  The caller orders the call after the work that produced every partial (on
 * other devices: an event or barrier across devices before this call) and keeps the partials
 * unchanged until the kernel has run.  Given the same partials in the same order every device
 * computes the same bits.  Errors: LIF_ERR_INVALID_ARG, LIF_ERR_ALIGNMENT, LIF_ERR_CUDA. */
#define LIF_MAX_PEERS 16
lif_status lif_sum_peer_outputs(const float* const* dev_partials, int32_t n_peers, float* dev_y,
                                size_t n_floats, void* stream);

/* One token through the layer: predict -> window update -> fetch -> sparse FFN (ffn_mode
 * selects the rows).  Two streams let the bundle fetch overlap the part of the FFN that does
 * not need the new rows; which of the two kernels runs on `fetch_stream` is the library's
 * choice (ordering is by events inside the call).  The compute stream ends up ordered after
 * everything, so consecutive calls on the same streams are safe.  Passing the same stream
 * twice runs the step serially. */
lif_status lif_decode_step(lif_layer* layer, const void* dev_x, float* dev_y,
                           void* compute_stream, void* fetch_stream);

/* One token through `n_layers` layers from host buffers: copies host_x (fp16
 * [n_streams][d_model], pinned) to dev_x, runs lif_decode_step on every layer in order with
 * layer l writing dev_y + l*n_streams*d_model, copies all outputs to host_y (fp32
 * [n_layers][n_streams][d_model], pinned) and synchronises compute_stream. */
lif_status lif_decode_token_host(lif_layer* const* layers, int32_t n_layers, const void* host_x,
                                 void* dev_x, float* dev_y, float* host_y,
                                 void* compute_stream, void* fetch_stream);

/* One token through `n_layers` layers as a CUDA graph.  lif_graph_capture records
 * lif_decode_step of every layer, in order, reading dev_x (fp16 [n_streams][d_model]) and with
 * layer l writing dev_y + l*n_streams*d_model, on two distinct non-default streams, and
 * instantiates the graph; nothing runs during capture.  Every size the kernels need is read
 * from device memory at run time, so one graph serves every token: put the token's input in
 * dev_x, then lif_graph_launch.  lif_graph_launch_host does that from pinned host buffers:
 * copies host_x in, launches, copies all layers' outputs to host_y (fp32
 * [n_layers][n_streams][d_model]) and synchronises the stream.  The layers must outlive the
 * graph.  Launch overhead per kernel is several times lower than separate launches. */
typedef struct lif_graph lif_graph;
lif_status lif_graph_capture(lif_layer* const* layers, int32_t n_layers, void* dev_x,
                             float* dev_y, void* compute_stream, void* fetch_stream,
                             lif_graph** out);
lif_status lif_graph_launch(lif_graph* graph, void* stream);
lif_status lif_graph_launch_host(lif_graph* graph, const void* host_x, float* host_y,
                                 void* stream);
lif_status lif_graph_destroy(lif_graph* graph);

/* Device addresses of lists and state (valid for the layer's lifetime). */
lif_status lif_get_lists(lif_layer* layer, lif_lists* host_out);

/* Synchronises the device, then reports counts, cumulative traffic and the status word. */
lif_status lif_get_stats(lif_layer* layer, lif_stats* host_out);

/* Host copies of the window state (any pointer may be NULL): pointers[capacity],
 * slot_of[d_ff], last_active[d_ff], num_used[1].  Synchronises the device. */
lif_status lif_read_state(lif_layer* layer, int32_t* host_pointers, int32_t* host_slot_of,
                          int32_t* host_last_active, int32_t* host_num_used);

/* Checkpoint / resume of one layer's window.  A snapshot holds the bookkeeping of Section 3.3
 * (counters including the step, pointers, slot_of, last_active, bias), not the cached rows:
 * lif_restore copies it back and re-reads rows 0..num_used-1 from the host bundle store, so a
 * restored layer continues exactly as the snapshotted one would have.  Both synchronise the
 * device; the buffer is plain host memory of at least lif_snapshot_bytes() bytes and is only
 * valid for a layer of the same description.  lif_restore checks the buffer on the host
 * before anything reaches the device (counters in range, pointers and slot_of inverse maps of
 * each other over exactly num_used rows, free rows marked -1, stamps older than the step);
 * LIF_ERR_STATE: it does not describe a state of this layer, and the layer is left as it was. */
lif_status lif_snapshot_bytes(lif_layer* layer, size_t* out_bytes);
lif_status lif_snapshot(lif_layer* layer, void* host_buf, size_t bytes);
lif_status lif_restore(lif_layer* layer, const void* host_buf, size_t bytes);

/* Clears the sticky device status word. */
lif_status lif_clear_status(lif_layer* layer, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LIF_H */
