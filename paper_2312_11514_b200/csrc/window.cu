// Sliding-window neuron cache bookkeeping (Section 3.1 "The Sliding Window Technique" and
// Section 3.3 "Optimized Data Management in DRAM", items 1 and 2), plus cold-cache reset and
// the row moves that keep the used rows consecutive.
//
// The plan is integer work over n_active + num_used elements, so one 1024-thread CTA does it
// with ordered block-wide compactions (one packed prefix scan per pass; list order = index
// order, never atomics order):
//   A  count what would be deleted / loaded; refuse on overflow before touching anything
//   B  stamp last_active of the active neurons
//   C  deleted rows in ascending slot order; surviving tail rows in descending slot order
//   D  first freed slot <- last surviving row (pointers, slot_of, bias); clear the tail
//   E  new neurons in ascending id get rows num_kept, num_kept + 1, ...
//   F  slot lists for the FFN
// The 4*d_model-byte row copies of step D run in a second, grid-wide kernel.
//
// append_first applies the two operations of Section 3.3 in the other order: the new neurons are
// stacked at rows n, n + 1, ... first, then the deletions pull the last rows into the freed
// ones.  A new neuron that would be moved straight away is simply given the freed row as the
// place its bundle is written to: with e deleted and l new neurons, the r = min(e, l) last new
// neurons take the r lowest freed rows (lowest row <- highest id), the others stay stacked, and
// only the e - r freed rows left over are closed by moving old rows (those at or beyond
// n - (e - r)).  Row moves and bundle writes then never touch the same row.
#include "lif_internal.cuh"

namespace lif {
namespace {

// Three counters ride in one 64-bit scan, 21 bits each (d_ff < 2^21 is checked at creation).
typedef unsigned long long u64;
constexpr int kField = 21;
constexpr u64 kFieldMask = (1ull << kField) - 1;
__device__ __forceinline__ u64 pack3(int a, int b, int c) {
  return (u64)a | ((u64)b << kField) | ((u64)c << (2 * kField));
}
__device__ __forceinline__ int field(u64 v, int i) { return (int)((v >> (i * kField)) & kFieldMask); }

struct Scan {
  u64 warp_sums[kWindowThreads / 32];
};

// exclusive prefix of v over the block (thread order); *total = block sum
__device__ __forceinline__ u64 block_scan(u64 v, u64* total, Scan& sc) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  u64 inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    u64 n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) sc.warp_sums[warp] = inc;
  __syncthreads();
  u64 ws = sc.warp_sums[lane];   // 32 warps
  u64 winc = ws;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    u64 n = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += n;
  }
  const u64 base = __shfl_sync(0xffffffffu, winc - ws, warp);
  *total = __shfl_sync(0xffffffffu, winc, 31);
  __syncthreads();
  return base + inc - v;
}

struct WindowArgs {
  const int32_t* act;
  const int32_t* n_act;
  int32_t* counts;
  int32_t *pointers, *slot_of, *last_active;
  __half* bias;
  const __half* bias_up;
  int32_t *active_idx, *evict_ids, *evict_slots, *move_src, *move_dst, *load_ids, *load_slots,
      *active_slots, *hit_slots;
  int F, cap, k;
  int budget;             // 0 = off; else rows the cache may hold (Appendix C memory budget)
  // Speculative decoding (Section 4): the step holds consecutive tokens; the kept window ends
  // with token `keep` of the step (keep = 1, keep_tok = nullptr: ordinary single-token update).
  const int8_t* keep_tok; // [F] last kept token per neuron, -1 if active only in later tokens
  int keep;
  int append_first;       // stack the new neurons before deleting (see the header of this file)
  int release_early;      // release the dependent kernel before this kernel's own wait
  unsigned long long bundle_bytes;
};

// Memory-budgeted window (Appendix C, Persimmon 8B / Phi-2): hist[a] = cached rows that are not
// active now and were last active a steps ago (a = 1 .. k, older ones in bin k).  Returns the
// widest window k' <= k for which the rows kept plus the rows to load fit `limit`, at least 1.
// Stamp of an active neuron: the time of the last kept token in which it is active (its old
// stamp if it is active only beyond the kept token), but never below the oldest stamp still
// inside the window that ends at t_end: this step does not delete it, the next one may.
__device__ __forceinline__ int active_stamp(const WindowArgs& a, int id, int t, int t_end) {
  if (!a.keep_tok) return t;
  const int j = a.keep_tok[id];
  return max(j >= 0 ? t + j : a.last_active[id], t_end - a.k + 1);
}

constexpr int kMaxBudgetWindow = 32;
constexpr int kSegRegs = 12;    // general path: cached rows per thread kept in registers
constexpr int kActRegs = 8;     // and active-list entries per thread
__device__ __forceinline__ int widest_window_that_fits(const int* hist, int k, int n, int n_load,
                                                       int limit) {
  int evicted = 0;          // rows deleted under window kk = sum of hist[a], a >= kk
  int kk = k;
  for (; kk >= 1; --kk) {
    evicted += hist[kk];
    if (n - evicted + n_load <= limit) break;
  }
  return kk < 1 ? 1 : kk;
}

// General path: any cache size, active list read from memory.
__device__ void window_update_generic(const WindowArgs& a, Scan& sc) {
  const int tid = threadIdx.x;
  const int n = a.counts[LIF_CNT_NUM_USED];
  const int t = a.counts[LIF_CNT_STEP];
  const int na = *a.n_act;
  const int t_end = t + a.keep - 1;   // the kept window ends at this token
  u64 tot;
  int bad = (na < 0 || na > a.F) ? 1 : 0;
  // a predictor input that never arrived left an incomplete active set: no update from it
  const int stale_input = a.counts[LIF_CNT_STATUS] == LIF_ERR_TIMEOUT;
  int k_eff = a.k;
  if (a.budget > 0) {
    // age histogram of the cached rows, minus those that are active again now
    __shared__ int hist[kMaxBudgetWindow + 1];
    __shared__ int loads;
    if (tid <= kMaxBudgetWindow) hist[tid] = 0;
    if (tid == 0) loads = 0;
    __syncthreads();
    if (!bad) {
      int c = 0;
      for (int q = tid; q < na; q += kWindowThreads) {
        const int id = a.act[q];
        if (id < 0 || id >= a.F) continue;
        if (a.slot_of[id] < 0) ++c;
        else atomicSub(&hist[min(a.k, max(1, t_end - a.last_active[id]))], 1);
      }
      if (c) atomicAdd(&loads, c);
      for (int s = tid; s < n; s += kWindowThreads)
        atomicAdd(&hist[min(a.k, max(1, t_end - a.last_active[a.pointers[s]]))], 1);
    }
    __syncthreads();
    k_eff = widest_window_that_fits(hist, a.k, n, loads, min(a.cap, a.budget));
    __syncthreads();
  }
  const int limit = a.budget > 0 ? min(a.cap, a.budget) : a.cap;
  const int stale_before = t_end - k_eff;   // last_active <= stale_before: outside the window

  // Register path: when a thread's run of cached rows and its run of the active list are
  // short (kSegRegs rows, kActRegs list entries), their ids are read once, and every pass below
  // issues its dependent loads (stamp, slot) for the whole run together instead of one entry
  // at a time between stores.  Same decisions, same lists.
  const int seg = (n + kWindowThreads - 1) / kWindowThreads;
  const int s0 = min(n, tid * seg), s1 = min(n, s0 + seg);
  const int na_ok = bad ? 0 : na;
  const int qseg = (na_ok + kWindowThreads - 1) / kWindowThreads;
  const int q0 = min(na_ok, tid * qseg), q1 = min(na_ok, q0 + qseg);
  const bool in_regs = seg <= kSegRegs && qseg <= kActRegs;     // uniform over the CTA
  int row_id[kSegRegs], act_id[kActRegs];
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) row_id[j] = s0 + j < s1 ? a.pointers[s0 + j] : 0;
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) act_id[j] = q0 + j < q1 ? a.act[q0 + j] : 0;
  }

  // ---- A: what would happen ------------------------------------------------------------
  int c_load = 0, c_back = 0, c_stale = 0;
  if (!bad && in_regs) {
    int so[kActRegs], la[kActRegs];
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) {
      so[j] = 0;
      la[j] = 0;
      if (q0 + j < q1) {
        if (act_id[j] < 0 || act_id[j] >= a.F) {
          bad = 1;
        } else {
          so[j] = a.slot_of[act_id[j]];
          la[j] = a.last_active[act_id[j]];
        }
      }
    }
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) {
      if (q0 + j < q1 && act_id[j] >= 0 && act_id[j] < a.F) {
        if (so[j] < 0) ++c_load;
        else if (la[j] <= stale_before) ++c_back;
      }
    }
    int ls[kSegRegs];
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) ls[j] = s0 + j < s1 ? a.last_active[row_id[j]] : 0;
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) c_stale += (s0 + j < s1 && ls[j] <= stale_before);
  } else if (!bad) {
    for (int q = tid; q < na; q += kWindowThreads) {
      const int id = a.act[q];
      if (id < 0 || id >= a.F) { bad = 1; continue; }
      if (a.slot_of[id] < 0) ++c_load;
      else if (a.last_active[id] <= stale_before) ++c_back;   // cached, stale, needed again
    }
    for (int s = tid; s < n; s += kWindowThreads)
      if (a.last_active[a.pointers[s]] <= stale_before) ++c_stale;
  }
  const int any_bad = __syncthreads_or(bad);
  block_scan(pack3(c_load, c_back, c_stale), &tot, sc);
  const int n_load = field(tot, 0);
  const int n_evict = field(tot, 2) - field(tot, 1);
  const int n_kept = n - n_evict;

  if (any_bad || stale_input || n_kept + n_load > limit) {
    if (tid == 0) {
      if (a.counts[LIF_CNT_STATUS] == LIF_OK)
        a.counts[LIF_CNT_STATUS] = any_bad ? LIF_ERR_INVALID_ARG : LIF_ERR_CAPACITY;
      a.counts[LIF_CNT_N_ACTIVE] = 0;
      a.counts[LIF_CNT_N_EVICT] = 0;
      a.counts[LIF_CNT_N_MOVES] = 0;
      a.counts[LIF_CNT_N_LOAD] = 0;
      a.counts[LIF_CNT_N_HITS] = 0;
      a.counts[LIF_CNT_NUM_USED_BEFORE] = n;
      a.counts[LIF_CNT_NUM_KEPT] = n;
    }
    return;
  }

  // ---- B: stamp --------------------------------------------------------------------------
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < kActRegs; ++j)
      if (q0 + j < q1) a.last_active[act_id[j]] = active_stamp(a, act_id[j], t, t_end);
  } else {
    for (int q = tid; q < na; q += kWindowThreads) {
      const int id = a.act[q];
      a.last_active[id] = active_stamp(a, id, t, t_end);
    }
  }
  __syncthreads();

  // ---- C: deleted rows (ascending slot) and surviving tail rows (descending slot) --------
  // Each thread owns a contiguous run of slots, so thread order is slot order.
  // r freed rows are taken by new neurons directly; the others are closed by old rows from
  // at or beyond `bound` (paper's order: r = 0, bound = n_kept)
  const int reuse = a.append_first ? min(n_evict, n_load) : 0;
  const int bound = n - (n_evict - reuse);
  int c_ev = 0, c_surv = 0;
  unsigned stale_rows = 0;                    // register path: bit j = row s0 + j is deleted
  if (in_regs) {
    int ls[kSegRegs];
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) ls[j] = s0 + j < s1 ? a.last_active[row_id[j]] : 0;
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) {
      if (s0 + j < s1) {
        const int f = ls[j] <= stale_before;
        stale_rows |= (unsigned)f << j;
        c_ev += f;
        c_surv += !f && s0 + j >= bound;
      }
    }
  } else {
    for (int s = s0; s < s1; ++s) {
      const int f = a.last_active[a.pointers[s]] <= stale_before;
      c_ev += f;
      c_surv += !f && s >= bound;
    }
  }
  u64 pre = block_scan(pack3(c_ev, 0, c_surv), &tot, sc);
  const int n_moves = field(tot, 2);          // surviving rows at or beyond the bound
  if (in_regs) {
    int p_ev = field(pre, 0), p_surv = field(pre, 2);
#pragma unroll
    for (int j = 0; j < kSegRegs; ++j) {
      const int s = s0 + j;
      if (s < s1) {
        if ((stale_rows >> j) & 1u) {
          a.evict_slots[p_ev] = s;
          a.evict_ids[p_ev] = row_id[j];
          ++p_ev;
        } else if (s >= bound) {
          a.move_src[n_moves - 1 - p_surv] = s;   // last survivor first
          ++p_surv;
        }
      }
    }
  } else {
    int p_ev = field(pre, 0), p_surv = field(pre, 2);
    for (int s = s0; s < s1; ++s) {
      const int id = a.pointers[s];
      const int f = a.last_active[id] <= stale_before;
      if (f) {
        a.evict_slots[p_ev] = s;
        a.evict_ids[p_ev] = id;
        ++p_ev;
      } else if (s >= bound) {
        a.move_src[n_moves - 1 - p_surv] = s;   // last survivor first
        ++p_surv;
      }
    }
  }
  __syncthreads();

  // ---- D: apply deletes to the bookkeeping ------------------------------------------------
  for (int j = tid; j < n_evict; j += kWindowThreads) a.slot_of[a.evict_ids[j]] = -1;
  for (int j = tid; j < n_moves; j += kWindowThreads) {
    const int src = a.move_src[j], dst = a.evict_slots[reuse + j];
    const int id = a.pointers[src];
    a.move_dst[j] = dst;
    a.pointers[dst] = id;
    a.slot_of[id] = dst;
    a.bias[dst] = a.bias[src];
  }
  __syncthreads();
  for (int s = bound + tid; s < n; s += kWindowThreads) a.pointers[s] = -1;
  __syncthreads();

  // ---- E + F: rows for the neurons to bring in, and the slot lists -----------------------
  int c_l = 0;
  int so_now[kActRegs];
  __half bu[kActRegs];
  if (in_regs) {
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) {
      so_now[j] = 0;
      bu[j] = __half();
      if (q0 + j < q1) {
        so_now[j] = a.slot_of[act_id[j]];
        bu[j] = a.bias_up[act_id[j]];
      }
    }
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) c_l += (q0 + j < q1 && so_now[j] < 0);
  } else {
    for (int q = q0; q < q1; ++q) c_l += a.slot_of[a.act[q]] < 0;
  }
  pre = block_scan(pack3(c_l, (q1 - q0) - c_l, 0), &tot, sc);
  if (in_regs) {
    int p_l = field(pre, 0), p_h = field(pre, 1);
#pragma unroll
    for (int j = 0; j < kActRegs; ++j) {
      const int q = q0 + j;
      if (q < q1) {
        const int id = act_id[j];
        int sl = so_now[j];
        if (sl < 0) {
          sl = p_l < n_load - reuse ? bound + p_l : a.evict_slots[n_load - 1 - p_l];
          a.load_ids[p_l] = id;
          a.load_slots[p_l] = sl;
          a.slot_of[id] = sl;
          a.pointers[sl] = id;
          a.bias[sl] = bu[j];
          ++p_l;
        } else {
          a.hit_slots[p_h++] = sl;
        }
        a.active_slots[q] = sl;
        if (a.active_idx != a.act) a.active_idx[q] = id;
      }
    }
  } else {
    int p_l = field(pre, 0), p_h = field(pre, 1);
    for (int q = q0; q < q1; ++q) {
      const int id = a.act[q];
      int s = a.slot_of[id];
      if (s < 0) {
        // stacked new neurons keep rows bound, bound + 1, ...; the last `reuse` of them take
        // the freed rows, lowest row <- highest id
        s = p_l < n_load - reuse ? bound + p_l : a.evict_slots[n_load - 1 - p_l];
        a.load_ids[p_l] = id;
        a.load_slots[p_l] = s;
        a.slot_of[id] = s;
        a.pointers[s] = id;
        a.bias[s] = a.bias_up[id];
        ++p_l;
      } else {
        a.hit_slots[p_h++] = s;
      }
      a.active_slots[q] = s;
      if (a.active_idx != a.act) a.active_idx[q] = id;
    }
  }
  if (tid == 0) {
    a.counts[LIF_CNT_N_ACTIVE] = na;
    a.counts[LIF_CNT_N_EVICT] = n_evict;
    a.counts[LIF_CNT_N_MOVES] = n_moves;
    a.counts[LIF_CNT_N_LOAD] = n_load;
    a.counts[LIF_CNT_N_HITS] = na - n_load;
    a.counts[LIF_CNT_NUM_USED_BEFORE] = n;
    a.counts[LIF_CNT_NUM_KEPT] = n_kept;
    a.counts[LIF_CNT_NUM_USED] = n_kept + n_load;
    a.counts[LIF_CNT_STEP] = t + a.keep;
    a.counts[LIF_CNT_K_EFF] = k_eff;
    unsigned long long* totals = reinterpret_cast<unsigned long long*>(a.counts + CNT_TOTALS);
    totals[0] += (unsigned long long)n_load * a.bundle_bytes;
    totals[1] += (unsigned long long)n_moves;
    totals[2] += (unsigned long long)na;
    totals[3] += (unsigned long long)(n_kept + n_load);
  }
}

__global__ void __launch_bounds__(kWindowThreads) window_update_kernel(WindowArgs a) {
  __shared__ Scan sc;
  if (a.release_early) pdl_trigger();     // see window_plan_kernel
  pdl_wait();
  if (!a.release_early) pdl_trigger();
  window_update_generic(a, sc);
}

// Fast path of the decode step: consumes the predictor's bit mask directly (the predictor then
// skips its own compaction) and keeps each thread's few slots and active neurons in registers,
// so the whole update is three dependent memory round trips (mask + counters; slot_of /
// pointers / biases; last_active of the cached neurons), three packed scans and the writes.
// Needs: at most kWindowThreads mask words, num_used <= kPlanSlots * kWindowThreads, at most
// kPlanBits active neurons per mask word.  Otherwise the CTA compacts the mask into the list
// and runs the general path.
constexpr int kPlanSlots = 4;
constexpr int kPlanBits = 12;
constexpr int kPlanMaxRows = kPlanSlots * kWindowThreads;

__global__ void __launch_bounds__(kWindowThreads)
window_plan_kernel(WindowArgs a, const uint32_t* __restrict__ mask_words, int nwords,
                   int32_t* n_act_out) {
  __shared__ Scan sc;
  __shared__ uint32_t bits[kWindowThreads];
  __shared__ int holes[kPlanMaxRows];
  __shared__ int newslot[kPlanMaxRows];
  const int tid = threadIdx.x;
  // Inside a decode step whose fetch kernel watches the predictor (kEarlyWatch) the kernel behind
  // this one is released at once: every kernel of the library waits for its predecessor's
  // completion before it touches that kernel's output, and the fetch kernel uses the time to
  // become resident and to watch the predictor finish.  Otherwise the release follows this
  // kernel's own wait, which is what lets a dependent read lists or masks ahead of its wait
  // (kEarlyLists, kEarlyMask).
  if (a.release_early) pdl_trigger();
  // The window state was last written by this layer's previous step, which is complete before
  // the predictor of this step even starts: the slot side of the bookkeeping (row -> neuron,
  // row bias, each cached neuron's stamp: three dependent round trips) is read before the
  // dependency wait and overlaps the predictor's tail.  Only the mask waits.
  const int n = a.counts[LIF_CNT_NUM_USED];
  const int t = a.counts[LIF_CNT_STEP];
  const int t_end = t + a.keep - 1;   // the kept window ends at this token
  const int seg = (n + kWindowThreads - 1) / kWindowThreads;   // <= kPlanSlots on the fast path
  const int s0 = min(n, tid * seg);
  const int my_slots = min(n, s0 + seg) - s0;
  int pid[kPlanSlots], la[kPlanSlots];
  __half pb[kPlanSlots];
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j) {
    pid[j] = 0;
    pb[j] = __half();
    if (j < my_slots) {
      pid[j] = a.pointers[s0 + j];
      pb[j] = a.bias[s0 + j];
    }
  }
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j) la[j] = j < my_slots ? a.last_active[pid[j]] : 0;
  pdl_wait();
  if (!a.release_early) pdl_trigger();
  const uint32_t w = tid < nwords ? mask_words[tid] : 0u;
  const int stale_input = a.counts[LIF_CNT_STATUS] == LIF_ERR_TIMEOUT;   // see the general path
  const int cnt = __popc(w);
  bits[tid] = w;
  u64 tot;
  const int q_base = field(block_scan(pack3(cnt, 0, 0), &tot, sc), 0);   // also publishes bits[]
  const int na = field(tot, 0);
  const int fast = __syncthreads_and(n <= kPlanMaxRows && cnt <= kPlanBits);
  if (!fast) {
    // compact the mask into the ascending list, then take the general path
    uint32_t m = w;
    for (int q = q_base; m; ++q, m &= m - 1) a.active_idx[q] = tid * 32 + __ffs(m) - 1;
    if (tid == 0) *n_act_out = na;
    __syncthreads();
    WindowArgs g = a;
    g.act = a.active_idx;
    g.n_act = n_act_out;
    window_update_generic(g, sc);
    return;
  }

  // ---- second round trip after the wait: by neuron id (mine: the bits of w) -------------------
  int so[kPlanBits];
  __half bu[kPlanBits];
  {
    uint32_t m = w;
#pragma unroll
    for (int i = 0; i < kPlanBits; ++i) {
      so[i] = 0;
      bu[i] = __half();
      if (m) {
        const int id = tid * 32 + __ffs(m) - 1;
        m &= m - 1;
        so[i] = a.slot_of[id];
        bu[i] = a.bias_up[id];
      }
    }
  }
  // ---- is each of my cached neurons still inside the window? -----------------------------------
  int age[kPlanSlots];          // steps since last active; 0 = active now
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j) {
    age[j] = 0;
    if (j < my_slots) {
      const int id = pid[j];
      const bool active_now = (bits[id >> 5] >> (id & 31)) & 1u;
      if (!active_now) age[j] = max(1, t_end - la[j]);
    }
  }
  int c_load = 0;
#pragma unroll
  for (int i = 0; i < kPlanBits; ++i) c_load += (i < cnt && so[i] < 0);
  int k_eff = a.k;
  if (a.budget > 0) {           // memory budget: shrink the window for this step if needed
    __shared__ int hist[kMaxBudgetWindow + 1];
    __shared__ int loads;
    if (tid <= kMaxBudgetWindow) hist[tid] = 0;
    if (tid == 0) loads = 0;
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kPlanSlots; ++j)
      if (age[j] > 0) atomicAdd(&hist[min(a.k, age[j])], 1);
    if (c_load) atomicAdd(&loads, c_load);
    __syncthreads();
    k_eff = widest_window_that_fits(hist, a.k, n, loads, min(a.cap, a.budget));
  }
  const int limit = a.budget > 0 ? min(a.cap, a.budget) : a.cap;
  unsigned evm = 0;             // bit j: slot s0 + j is deleted
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j)
    if (age[j] >= k_eff) evm |= 1u << j;
  u64 pre = block_scan(pack3(c_load, __popc(evm), cnt - c_load), &tot, sc);
  const int n_load = field(tot, 0), n_evict = field(tot, 1);
  const int n_kept = n - n_evict;
  int p_load = field(pre, 0), p_ev = field(pre, 1), p_hit = field(pre, 2);

  if (stale_input || n_kept + n_load > limit) {            // refuse before anything is changed
    if (tid == 0) {
      if (a.counts[LIF_CNT_STATUS] == LIF_OK) a.counts[LIF_CNT_STATUS] = LIF_ERR_CAPACITY;
      a.counts[LIF_CNT_N_ACTIVE] = 0;
      a.counts[LIF_CNT_N_EVICT] = 0;
      a.counts[LIF_CNT_N_MOVES] = 0;
      a.counts[LIF_CNT_N_LOAD] = 0;
      a.counts[LIF_CNT_N_HITS] = 0;
      a.counts[LIF_CNT_NUM_USED_BEFORE] = n;
      a.counts[LIF_CNT_NUM_KEPT] = n;
    }
    return;
  }
  // freed rows taken by new neurons directly, and where the rows that must move begin
  // (paper's order: none, num_kept; see the header of this file)
  const int reuse = a.append_first ? min(n_evict, n_load) : 0;
  const int bound = n - (n_evict - reuse);
  int c_surv = 0;
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j)
    if (j < my_slots) c_surv += !((evm >> j) & 1u) && (s0 + j) >= bound;
  pre = block_scan(pack3(c_surv, 0, 0), &tot, sc);
  const int n_moves = field(tot, 0);          // surviving rows at or beyond the bound
  int p_surv = field(pre, 0);

  // ---- writes ---------------------------------------------------------------------------------
  {
    uint32_t m = w;
    for (; m; m &= m - 1) {                                                    // stamp
      const int id = tid * 32 + __ffs(m) - 1;
      a.last_active[id] = active_stamp(a, id, t, t_end);
    }
  }
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j)
    if (j < my_slots && ((evm >> j) & 1u)) {                                     // deleted rows
      const int s = s0 + j;
      a.evict_ids[p_ev] = pid[j];
      a.slot_of[pid[j]] = -1;
      holes[p_ev++] = s;                                 // freed rows, ascending
    }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < kPlanSlots; ++j)
    if (j < my_slots) {
      const int s = s0 + j;
      if (!((evm >> j) & 1u) && s >= bound) {          // surviving tail row: last one first
        const int jm = n_moves - 1 - p_surv++;
        const int dst = holes[reuse + jm];
        a.move_src[jm] = s;
        a.move_dst[jm] = dst;
        a.pointers[dst] = pid[j];
        a.slot_of[pid[j]] = dst;
        a.bias[dst] = pb[j];
        newslot[s - bound] = dst;
      }
      if (s >= n_kept + n_load) a.pointers[s] = -1;    // tail beyond the rows to be loaded
    }
  __syncthreads();
  {
    uint32_t m = w;
    int q = q_base;
#pragma unroll
    for (int i = 0; i < kPlanBits; ++i)
      if (i < cnt) {
        const int id = tid * 32 + __ffs(m) - 1;
        m &= m - 1;
        int s = so[i];
        if (s < 0) {                                     // bring in: stacked rows, or freed ones
          s = p_load < n_load - reuse ? bound + p_load : holes[n_load - 1 - p_load];
          a.load_ids[p_load] = id;
          a.load_slots[p_load] = s;
          ++p_load;
          a.slot_of[id] = s;
          a.pointers[s] = id;
          a.bias[s] = bu[i];
        } else {
          if (s >= bound) s = newslot[s - bound];        // it was moved into a freed row
          a.hit_slots[p_hit++] = s;
        }
        a.active_slots[q] = s;
        a.active_idx[q] = id;
        ++q;
      }
  }
  if (tid == 0) {
    *n_act_out = na;
    a.counts[LIF_CNT_N_ACTIVE] = na;
    a.counts[LIF_CNT_N_EVICT] = n_evict;
    a.counts[LIF_CNT_N_MOVES] = n_moves;
    a.counts[LIF_CNT_N_LOAD] = n_load;
    a.counts[LIF_CNT_N_HITS] = na - n_load;
    a.counts[LIF_CNT_NUM_USED_BEFORE] = n;
    a.counts[LIF_CNT_NUM_KEPT] = n_kept;
    a.counts[LIF_CNT_NUM_USED] = n_kept + n_load;
    a.counts[LIF_CNT_STEP] = t + a.keep;
    a.counts[LIF_CNT_K_EFF] = k_eff;
    unsigned long long* totals = reinterpret_cast<unsigned long long*>(a.counts + CNT_TOTALS);
    totals[0] += (unsigned long long)n_load * a.bundle_bytes;
    totals[1] += (unsigned long long)n_moves;
    totals[2] += (unsigned long long)na;
    totals[3] += (unsigned long long)(n_kept + n_load);
  }
}

// Row moves of step D: cache row move_src[j] -> row move_dst[j].  Sources lie at or beyond
// num_kept (append_first: the bound above which old rows must move), destinations below it, so
// the copies never overlap.
__global__ void __launch_bounds__(kThreads)
move_rows_kernel(uint4* __restrict__ cache, const int32_t* __restrict__ move_src,
                 const int32_t* __restrict__ move_dst, const int32_t* __restrict__ counts,
                 int row_vec, int release_early) {
  // release_early: the kernel behind is the fetch kernel in its watching form, which reads
  // nothing of this step's lists or rows before its own wait (see window_plan_kernel)
  if (release_early) pdl_trigger();
  pdl_wait();
  if (!release_early) pdl_trigger();
  const int n = counts[LIF_CNT_N_MOVES];
  for (int j = blockIdx.x; j < n; j += gridDim.x) {
    const uint4* src = cache + (size_t)move_src[j] * row_vec;
    uint4* dst = cache + (size_t)move_dst[j] * row_vec;
#pragma unroll 4
    for (int v = threadIdx.x; v < row_vec; v += kThreads) dst[v] = src[v];
  }
}

__global__ void __launch_bounds__(kThreads)
reset_kernel(int32_t* counts, int32_t* pointers, int32_t* slot_of, int32_t* last_active,
             uint32_t* mask_words, unsigned long long* new_mask_words, int n_mask, int n_new, int F,
             int cap) {
  const int i = blockIdx.x * kThreads + threadIdx.x;
  const int stride = gridDim.x * kThreads;
  // predictor runs are numbered from 1: no entry of new_mask_words carries a number in use
  for (int j = i; j < LIF_CNT_LEN; j += stride) counts[j] = j == CNT_PREDICTOR_RUN ? 1 : 0;
  for (int j = i; j < cap; j += stride) pointers[j] = -1;
  for (int j = i; j < F; j += stride) {
    slot_of[j] = -1;
    last_active[j] = kNever;
  }
  for (int j = i; j < n_mask; j += stride) mask_words[j] = 0;
  for (int j = i; j < n_new; j += stride) new_mask_words[j] = 0ull;
}

}  // namespace

cudaError_t launch_reset(lif_layer* L, cudaStream_t st) {
  const lif_layer_desc& D = L->desc;
  const int n_mask = (D.d_ff + kLogitTile - 1) / kLogitTile * (kLogitTile / 32);
  reset_kernel<<<64, kThreads, 0, st>>>(L->counts, L->pointers, L->slot_of, L->last_active,
                                        L->mask_words, L->new_mask_words, n_mask,
                                        new_mask_entries(D), D.d_ff, D.capacity);
  return cudaGetLastError();
}

static WindowArgs window_args(lif_layer* L, const int32_t* act, const int32_t* n_act) {
  const lif_layer_desc& D = L->desc;
  WindowArgs a;
  a.act = act;
  a.n_act = n_act;
  a.counts = L->counts;
  a.pointers = L->pointers;
  a.slot_of = L->slot_of;
  a.last_active = L->last_active;
  a.bias = L->bias;
  a.bias_up = (const __half*)D.dev_bias_up;
  a.active_idx = L->active_idx;
  a.evict_ids = L->evict_ids;
  a.evict_slots = L->evict_slots;
  a.move_src = L->move_src;
  a.move_dst = L->move_dst;
  a.load_ids = L->load_ids;
  a.load_slots = L->load_slots;
  a.active_slots = L->active_slots;
  a.hit_slots = L->hit_slots;
  a.F = D.d_ff;
  a.cap = D.capacity;
  a.k = D.window_k;
  a.budget = D.budget_rows;
  a.keep_tok = D.spec_keep > 0 ? L->keep_tok : nullptr;
  a.keep = D.spec_keep > 0 ? D.spec_keep : 1;
  a.bundle_bytes = 2ull * row_elems(D);
  a.append_first = D.append_first;
  a.release_early = L->watch_chain;
  return a;
}

cudaError_t launch_moves(lif_layer* L, cudaStream_t st, cudaEvent_t* ev, bool release_early) {
  const lif_layer_desc& D = L->desc;
  cudaError_t e;
  if (ev) tm_record(ev[3], st);
  e = launch_k(move_rows_kernel, dim3(L->move_grid), dim3(kThreads), 0, st, L->use_pdl,
               (uint4*)D.dev_cache, (const int32_t*)L->move_src, (const int32_t*)L->move_dst,
               (const int32_t*)L->counts, row_elems(D) / 8, release_early ? 1 : 0);
  if (ev) tm_record(ev[4], st);
  return e;
}

cudaError_t launch_window(lif_layer* L, const int32_t* act, const int32_t* n_act,
                          cudaStream_t st, cudaEvent_t* ev, bool with_moves) {
  cudaError_t e = launch_k(window_update_kernel, dim3(1), dim3(kWindowThreads), 0, st, L->use_pdl,
                           window_args(L, act, n_act));
  return (e != cudaSuccess || !with_moves) ? e : launch_moves(L, st, ev, L->watch_chain != 0);
}

bool window_plan_supported(const lif_layer_desc& D) {
  return (D.d_ff + kLogitTile - 1) / kLogitTile * (kLogitTile / 32) <= kWindowThreads;
}

// Window update straight from the predictor's bit mask (see window_plan_kernel).
cudaError_t launch_window_plan(lif_layer* L, cudaStream_t st, cudaEvent_t* ev, bool with_moves) {
  const lif_layer_desc& D = L->desc;
  const int nwords = (D.d_ff + kLogitTile - 1) / kLogitTile * (kLogitTile / 32);
  cudaError_t e = launch_k(window_plan_kernel, dim3(1), dim3(kWindowThreads), 0, st, L->use_pdl,
                           window_args(L, L->active_idx, L->n_tmp), (const uint32_t*)L->mask_words,
                           nwords, (int32_t*)L->n_tmp);
  return (e != cudaSuccess || !with_moves) ? e : launch_moves(L, st, ev, L->watch_chain != 0);
}

}  // namespace lif
