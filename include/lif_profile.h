/*
 * lif_profile.h — tuning knobs and profiling aids of liblif.so.  Nothing here is part of the
 * method (arXiv 2312.11514 has no counterpart to any of it): the knobs change launch shapes
 * and never results beyond the order of floating-point partial sums; the aids time kernels
 * and the host link.  The calls of the method itself are in lif.h.
 */
#ifndef LIF_PROFILE_H
#define LIF_PROFILE_H

#include "lif.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Launch-shape knobs (defaults in parentheses); they change speed, never results beyond the
 * order of floating-point partial sums.  Set them before capturing a graph. */
enum {
  LIF_TUNE_DEPENDENT_LAUNCH = 0, /* (1) programmatic dependent launch along the compute stream */
  LIF_TUNE_SPLIT_FFN = 1,        /* (1) lif_decode_step runs the FFN of already-cached rows
                                    while the fetch copies, then the FFN of the new rows */
  LIF_TUNE_FETCH_CTAS = 2,       /* (SM count) CTAs of the fetch kernel, 1..4096 */
  LIF_TUNE_FFN_CTAS = 3,         /* (SM count) CTAs of the sparse-FFN kernel, 1..256 */
  LIF_TUNE_FFN_STAGES = 4,       /* (as many as fit, at most 16) bundles in flight per CTA;
                                    fewer stages let several CTAs share an SM */
  LIF_TUNE_BATCHED_COLUMN_PARTS = 5, /* (fewest that fit) column parts of the multi-stream FFN's
                                    down-projection kernel, 1..16 */
  LIF_TUNE_BATCHED_UP_TWO_CTAS = 7, /* (0) multi-stream FFN, up-projection kernel: two light CTAs
                                    per SM instead of one with a deep ring */
  LIF_TUNE_FUSED_PLAN = 6,       /* (1 when d_ff <= 32768) lif_decode_step: the window update
                                    reads the predictor's bit mask instead of its index list */
  LIF_TUNE_FUSED_FETCH_FFN = 8,  /* (1) lif_decode_step, one stream, with LIF_TUNE_SPLIT_FFN: the
                                    fetch kernel also adds the FFN terms of the rows it brings
                                    in (needs fetch CTAs = FFN CTAs, bundles of two vectors) */
  LIF_TUNE_WAIT_POLLS = 9,       /* (2^22) test aid: poll limit of the FIRST wait on each bulk
                                    copy in the sparse-FFN kernels, >= 0 (0: give up without
                                    polling).  When it runs out the CTA sets LIF_ERR_TIMEOUT,
                                    then waits for its copies with the full limit before it
                                    returns, so 0 makes the error path run with nothing left in
                                    flight */
  LIF_TUNE_EARLY_FETCH = 10      /* (1) lif_decode_step where the fetch is a kernel of its own
                                    (several input streams, three-vector bundles): it runs on
                                    the compute stream directly behind the window kernel, is
                                    resident while the predictor still runs and issues its first
                                    host loads from the predictor's masks; 0: it waits for the
                                    window kernel's lists on the fetch stream */
};
lif_status lif_set_tuning(lif_layer* layer, int32_t key, int32_t value);

/* Phases timed by lif_timing_* (one CUDA event pair each, inside lif_decode_step). */
enum {
  LIF_PHASE_PREDICT_Z = 0,      /* x.A partial sums */
  LIF_PHASE_PREDICT_SCORES = 1, /* scores, threshold, compaction */
  LIF_PHASE_WINDOW = 2,         /* window bookkeeping kernel */
  LIF_PHASE_MOVES = 3,          /* row moves */
  LIF_PHASE_FETCH = 4,          /* bundle fetch (on the fetch stream) */
  LIF_PHASE_FFN = 5,            /* sparse FFN gather kernel(s) */
  LIF_PHASE_FFN_SUM = 6,        /* partial-sum kernel(s) */
  LIF_PHASE_LEN = 8
};

/* Profiling aid: with n_steps > 0, the next n_steps calls of lif_decode_step record CUDA
 * events around every kernel (host-side event objects, no device memory); n_steps = 0 turns
 * it off and frees the events.  lif_timing_read synchronises the device and returns, per
 * phase, the summed device time in microseconds over the steps recorded since enabling. */
lif_status lif_timing_enable(lif_layer* layer, int32_t n_steps);
lif_status lif_timing_read(lif_layer* layer, float* host_us_sums /* [LIF_PHASE_LEN] */,
                           int32_t* host_n_steps);

/* Profiling aid: enqueue exactly one kernel of the decode step, with the launch shape
 * lif_decode_step uses, on the layer's current lists (valid after a completed step; these
 * kernels do not change the window state, so they can be replayed).  dev_x as for
 * lif_decode_step; dev_y is written only by LIF_KERNEL_FFN_SUM.  n_streams must be 1. */
enum {
  LIF_KERNEL_PREDICT_Z = 0,  /* LIF_ERR_STATE with LIF_GATE_RESIDENT (no first stage) */
  LIF_KERNEL_PREDICT_SCORES = 1, /* LIF_GATE_RESIDENT: the gate-projection kernel */
  LIF_KERNEL_FETCH = 2,      /* re-copies this step's new bundles (and, where the decode step
                                fuses it, recomputes their FFN partials) */
  LIF_KERNEL_FFN_ACTIVE = 3, /* sparse FFN kernel over all active rows */
  LIF_KERNEL_FFN_HITS = 4,   /* ... over the active rows that were already cached */
  LIF_KERNEL_FFN_NEW = 5,    /* ... over the rows brought in this step */
  LIF_KERNEL_FFN_SUM = 6,    /* partial-sum kernel over the hits + new partials */
  LIF_KERNEL_FFN_CACHE = 7   /* sparse FFN kernel over every cached row, [0, num_used): what
                                Section 3.3 item 3 writes (matrix[:num_rows]) */
};
lif_status lif_profile_launch(lif_layer* layer, int32_t kernel, const void* dev_x, float* dev_y,
                              void* stream);

/* Bandwidth probe for the host link: a kernel reads `bytes` of mapped pinned host memory
 * into device memory with the same access pattern as lif_fetch_bundles (chunk_bytes-sized
 * pieces; chunk_bytes a multiple of 16, bytes a multiple of chunk_bytes).  Enqueue only. */
lif_status lif_probe_host_read(const void* host_src, void* dev_dst, size_t bytes,
                               size_t chunk_bytes, void* stream);

/* Reference point for kernels that read a few megabytes per launch: a kernel that does nothing
 * but read `bytes` (a multiple of 16) of device memory with 16-byte loads from ctas_per_sm CTAs
 * on every SM (1..8), launched with (dependent_launch != 0) or without the programmatic
 * dependent-launch attribute the decode step's kernels use.  dev_sink: 16 bytes of device memory
 * that are (practically never) written.  Enqueue only. */
lif_status lif_probe_device_read(const void* dev_src, size_t bytes, void* dev_sink,
                                 int32_t ctas_per_sm, int32_t dependent_launch, void* stream);

/* Reference point for the kernels that stream rows through a ring of bulk copies: every CTA
 * (ctas_per_sm on every SM, 256 threads) streams an equal share of `bytes` of device memory in
 * pieces of chunk_bytes (multiple of 16) through a shared-memory ring of `stages` stages,
 * refilled refill_group stages at a time (stages a multiple of it, at most 256 per group) with
 * one mbarrier per group and bounded waits.  threads_every = 0: every stage is filled by one bulk copy; n > 0: every n-th
 * stage is filled by 16-byte asynchronous copies of all threads instead.  The data is only
 * touched (4 bytes per thread and stage).  dev_timeouts: int32 on the device, incremented by a
 * CTA whose wait ran out (it then lets its copies land and leaves).  stages * (chunk_bytes + 8)
 * must fit the shared memory of a CTA.  Enqueue only. */
lif_status lif_probe_bulk_ring(const void* dev_src, size_t bytes, uint32_t chunk_bytes,
                               int32_t stages, int32_t refill_group, int32_t ctas_per_sm,
                               int32_t threads_every, void* dev_sink, int32_t* dev_timeouts,
                               void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LIF_PROFILE_H */
