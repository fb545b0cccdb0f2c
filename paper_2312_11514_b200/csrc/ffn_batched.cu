// Sparse FFN for several decode streams sharing one layer (Section 3.3 item 3 applied to S
// inputs at once): over the gathered rows the computation is a dense contraction,
//   H[q][s] = relu(<M[slot_q, :d], x[s]> + bias[slot_q])        (up halves,   K = d_model)
//   Y[s][m] = b_down[m] + sum_q H[q][s] * M[slot_q, d + m]       (down halves, K = rows)
// so it runs on tensor cores (mma.sync m16n8k16, fp16 operands, fp32 accumulate) while every
// bundle half is still read from HBM exactly once:
//   phase A: CTAs own (row partition, K slice); that slice of the up halves streams through a
//            ring of shared-memory stages (one bulk copy per row), 16 rows per MMA as the A
//            operand; the same slice of x (S x d, fp16) stays in shared memory as the B operand;
//            the 8 warps split the slice and fold through shared memory.  Output: partial
//            pre-activations per K slice (slice 0 carries the bias).
//   phase B: CTAs own (row partition, column part); the down halves of the part stream through
//            the ring, 16 rows per MMA k-step; H = relu(sum of the K-slice partials), split into
//            fp16 high + low parts (so the product keeps fp32 accuracy), is the B operand; each
//            warp keeps its column tiles' accumulators in registers for the whole kernel.  H is
//            scaled by a power of two before the split (the largest magnitude seen so far maps
//            near 2^10; accumulators are rescaled exactly when it grows), so the result does not
//            depend on where the activations sit in fp16's narrow exponent range.
// Partition partials are added in a fixed order by the partial-sum kernel.  Bound: HBM.
// Gated layers (Appendix C, Llama 2): with the gate row in the bundle, phase A runs twice (gate
// rows with the bias, then up rows) and phase B uses H = act(gate) * up; with the gate
// projection resident, phase A contracts the up rows and phase B takes the gate value of each
// row's neuron from the predictor's score array.
#include "lif_internal.cuh"

namespace lif {
namespace {

constexpr int kPad = 16;                  // bytes added to every shared row: conflict-free ldmatrix
constexpr int kGroupA = 16;               // rows per MMA in phase A (M = 16)
// One mbarrier per group of 16 ring stages (the first stage's): arrival count 16, one arrival
// per stage — with the stage's byte count where a row is copied, plain where the list has ended.
constexpr int kGroup = 16;
__device__ __forceinline__ uint64_t* group_bar(uint64_t* bars, int stage, int group = kGroup) {
  return bars + (stage / group) * group;
}
constexpr int kMaxTilesPerWarp = 28;      // 16-column tiles per warp in phase B
constexpr int kRowCacheA = 512;           // rows per CTA whose slot and bias are preloaded (phase A)
constexpr int kRowCacheB = 256;           // rows per CTA whose slot is preloaded (phase B)

__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
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
  float* H;               // [ksplit][h_stride] fp32; entry [q][8], position-indexed
  float* y_partial;       // [partitions][S][d]
  int32_t* status;
  int d, S, stages, parts, partitions, cols_per_part;
  int ksplit, k_per_split, up_partitions;   // phase A: K slices (columns, multiple of 16)
  int up_group;                             // phase A: rows per group (8 or 16; MMA M is 16)
  size_t h_stride;
  int act;                // LIF_ACT_*
  float act_thr;
  int row_elems;          // fp16 elements per cache row
  int vec_off;            // phase A: first element of the vector it contracts (gate or up row)
  int down_off;           // phase B: first element of the down column
  int add_bias;           // phase A: K slice 0 adds the row's bias
  int gate_mode;          // LIF_GATE_*
  int F;
  const float* H2;        // bundled gate: phase-A output of the up rows (H holds the gate rows)
  const float* gate_val;  // resident gate: [S][F] gate pre-activations by neuron id
  const int32_t* pointers;  // resident gate: row -> neuron id
  int rows;               // rows of `cache`: a slot outside [0, rows) is refused, not read
  unsigned wait_polls;    // poll limit of the first wait on each group of copies
};

// Cache row of list position q, or -1 when the list names a row outside the cache (such a row is
// never read: row 0 travels in its place and its activations are forced to zero).
__device__ __forceinline__ int row_slot(const BatchedArgs& a, int q, int base) {
  const int slot = a.slots ? a.slots[q] : base + q;
  return (slot < 0 || slot >= a.rows) ? -1 : slot;
}
// Row count as every kernel of this path clamps it: [0, rows].
__device__ __forceinline__ int row_count(const BatchedArgs& a) {
  const int n = *a.n;
  return n < 0 ? 0 : (n > a.rows ? a.rows : n);
}
// After a wait ran out: one more bounded chance for every copy still in flight to land in this
// CTA's shared memory (a barrier is re-polled with the parity of its current phase; one whose
// phase already completed returns at once).
__device__ __forceinline__ void drain_ring(uint64_t* bars, int stages, int group, int g,
                                           int groups_in_ring) {
  for (int k = 0; k < groups_in_ring; ++k) {
    const int gg = g + k;                              // groups g .. g + ring - 1 may be armed
    mbar_wait(bars + (gg % groups_in_ring) * group, (unsigned)(gg / groups_in_ring) & 1u);
  }
}

// ---- phase A: partial pre-activations  Hp[slice][q][s] = <Up[q, slice], x[s, slice]> (+ bias) --
__global__ void __launch_bounds__(kThreads, 2) ffn_batched_up_kernel(BatchedArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = a.d;
  const int ks = blockIdx.x % a.ksplit, prt = blockIdx.x / a.ksplit;
  const int k0 = ks * a.k_per_split;                    // first column of this K slice
  const int kcols = min(a.k_per_split, d - k0);
  const unsigned seg_bytes = 2u * kcols;
  const unsigned pitch = 2u * a.k_per_split + kPad;
  const int stages = a.stages;                          // multiple of the group size
  const int G = a.up_group;                             // rows per group: 8 or 16
  unsigned char* xs = smem;                                  // [8][pitch]
  unsigned char* rows = xs + 8 * (size_t)pitch;              // [stages][pitch]
  uint64_t* bars = reinterpret_cast<uint64_t*>(rows + (size_t)stages * pitch);
  float* bias_s = reinterpret_cast<float*>(bars + stages);   // [stages]
  float* red = bias_s + stages;                              // [8 warps][32 lanes][4]
  int* slot_all = reinterpret_cast<int*>(red + 8 * 32 * 4);  // [kRowCacheA]
  float* bias_all = reinterpret_cast<float*>(slot_all + kRowCacheA);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, G);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  pdl_wait();
  pdl_trigger();
  const int n = row_count(a);
  if (n != *a.n && blockIdx.x == 0 && tid == 0) atomicCAS(a.status, LIF_OK, LIF_ERR_INVALID_ARG);
  if (prt >= n) return;
  const int base = a.base ? *a.base : 0;
  const int P = a.up_partitions;
  const int my_cnt = (n - prt + P - 1) / P;             // rows q = prt + i * P
  __syncthreads();

  // Slots and biases of this CTA's rows go to shared memory once, so the group loop below has
  // no dependent global loads; the first copies are issued on the way.  Then the x slice
  // (streams beyond S are zero).
  // a refused row is remembered as a NaN bias: its pre-activations are written as zero
  const float kRefused = __int_as_float(0x7fc00000);
  for (int i = tid; i < min(my_cnt, kRowCacheA); i += kThreads) {
    int slot = row_slot(a, prt + i * P, base);
    const bool refused = slot < 0;
    if (refused) {
      atomicCAS(a.status, LIF_OK, LIF_ERR_INVALID_ARG);
      slot = 0;
    }
    slot_all[i] = slot;
    if (i < stages) {
      mbar_expect_tx(group_bar(bars, i, G), seg_bytes);
      bulk_g2s(rows + (size_t)i * pitch, a.cache + (size_t)slot * a.row_elems + a.vec_off + k0,
               seg_bytes, group_bar(bars, i, G));
    }
    const float b = refused ? kRefused
                            : ((ks == 0 && a.add_bias) ? __half2float(a.bias[slot]) : 0.f);
    bias_all[i] = b;
    if (i < stages) bias_s[i] = b;
  }
  for (int i = my_cnt + tid; i < stages; i += kThreads) mbar_arrive(group_bar(bars, i, G));
  {
    const int vec = kcols >> 3;
    for (int i = tid; i < 8 * vec; i += kThreads) {
      const int s = i / vec, c = i % vec;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (s < a.S) v = reinterpret_cast<const uint4*>(a.x + (size_t)s * d + k0)[c];
      *reinterpret_cast<uint4*>(xs + (size_t)s * pitch + (size_t)c * 16) = v;
    }
  }
  __syncthreads();

  const int ksteps = kcols >> 4;
  const int kper = (ksteps + 7) >> 3;
  const int k_begin = warp * kper, k_end = min(ksteps, k_begin + kper);
  const int gq = lane >> 2, tq = lane & 3;              // fragment coordinates
  const unsigned char* xb = xs + (size_t)gq * pitch + tq * 4;            // B: stream gq
  // A (16 rows x 16 columns): lane supplies row (lane % 8) + 8 * (lane / 8 % 2), columns
  // 8 * (lane / 16) of the k-step
  // (with 8-row groups the upper half of the tile repeats the lower one; its results are unused)
  const int a_row = (lane & 7) + (G == 16 ? ((lane >> 3) & 1) * 8 : 0);
  const int a_off = (lane >> 4) * 16;
  float* Hp = a.H + (size_t)ks * a.h_stride;
  int timed_out = 0;
  const int n_groups = (my_cnt + G - 1) / G;
  const int groups_in_ring = stages / G;
  for (int g = 0; g < n_groups; ++g) {
    const int st0 = (g % groups_in_ring) * G;
    const unsigned parity = (unsigned)(g / groups_in_ring) & 1u;
    const int valid = min(G, my_cnt - g * G);
    if (!mbar_wait(bars + st0, parity, a.wait_polls)) timed_out = 1;
    // D[row][stream] over this warp's part of the slice
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    const unsigned char* ab = rows + (size_t)(st0 + a_row) * pitch + a_off;
#pragma unroll 4
    for (int k = k_begin; k < k_end; ++k) {
      uint32_t af[4];
      ldmatrix_x4(af, ab + k * 32);
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(xb + k * 32);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(xb + k * 32 + 16);
      mma16816(c, af, b0, b1);
    }
    // c[0], c[1] = (row gq, streams 2*tq, 2*tq + 1); c[2], c[3] = row gq + 8; fold the 8 warps
    *reinterpret_cast<float4*>(red + (warp * 32 + lane) * 4) = make_float4(c[0], c[1], c[2], c[3]);
    if (__syncthreads_or(timed_out)) {
      if (tid == 0) {
        atomicCAS(a.status, LIF_OK, LIF_ERR_TIMEOUT);
        drain_ring(bars, stages, G, g, groups_in_ring);
      }
      __syncthreads();
      return;
    }
    if (tid < 8 * G) {
      const int r = tid >> 3, s = tid & 7;              // row in group, stream
      if (r < valid) {
        const int src = ((r & 7) * 4 + (s >> 1)) * 4 + (r >> 3) * 2 + (s & 1);
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[w * 128 + src];
        const int q = prt + (g * G + r) * P;
        const float b = bias_s[st0 + r];
        Hp[(size_t)q * 8 + s] = b == b ? v + b : 0.f;     // NaN marks a refused row
      }
    }
    __syncthreads();                                    // stages st0.. , bias_s and red are free
    // refill with the rows of group g + groups_in_ring
    if (tid < G) {
      const int i = (g + groups_in_ring) * G + tid;
      if (i < my_cnt) {
        const bool cached = i < kRowCacheA;
        int slot = cached ? slot_all[i] : row_slot(a, prt + i * P, base);
        const bool refused = slot < 0;
        if (refused) {
          atomicCAS(a.status, LIF_OK, LIF_ERR_INVALID_ARG);
          slot = 0;
        }
        mbar_expect_tx(bars + st0, seg_bytes);
        bulk_g2s(rows + (size_t)(st0 + tid) * pitch,
                 a.cache + (size_t)slot * a.row_elems + a.vec_off + k0, seg_bytes, bars + st0);
        bias_s[st0 + tid] =
            cached ? bias_all[i]
                   : (refused ? kRefused
                              : ((ks == 0 && a.add_bias) ? __half2float(a.bias[slot]) : 0.f));
      } else {
        mbar_arrive(bars + st0);
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
  int* slot_all = reinterpret_cast<int*>(h_lo + 128);                  // [kRowCacheB]
  // per group parity: max |H| of the four warps that load H
  float (*gmax)[4] = reinterpret_cast<float (*)[4]>(slot_all + kRowCacheB);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int i = 0; i < stages; ++i) mbar_init(bars + i, kGroup);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // This kernel always follows ffn_batched_up_kernel on its stream and depends on it only
  // through H.  Rows, slots and counters were final before that kernel passed its own
  // dependency wait (it signals its dependents only afterwards), so they are read, and the
  // first copies issued, before the wait below: the prologue overlaps the up kernel's tail.
  const int n = row_count(a);
  const int base = a.base ? *a.base : 0;
  const int P = a.partitions;
  const int my_cnt = prt < n ? (n - prt + P - 1) / P : 0;       // rows q = prt + i * P
  // Padded k-steps (rows past the end of the list) multiply by H = 0 and need finite operands.
  // Once the ring has been filled they hold earlier rows' weights; a list shorter than the
  // ring leaves stages never written, so those are zeroed first.
  if (my_cnt < stages)
    for (size_t i = (size_t)tid * 16; i < (size_t)stages * pitch; i += kThreads * 16)
      *reinterpret_cast<uint4*>(rows + i) = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  const size_t col_off = (size_t)a.down_off + col0;

  // (a refused row was reported by the up kernel and has H = 0: row 0 stands in for it)
  for (int i = tid; i < min(my_cnt, kRowCacheB); i += kThreads) {   // slots once, first copies
    const int slot = max(0, row_slot(a, prt + i * P, base));
    slot_all[i] = slot;
    if (i < stages) {
      mbar_expect_tx(group_bar(bars, i), seg_bytes);
      bulk_g2s(rows + (size_t)i * pitch, a.cache + (size_t)slot * a.row_elems + col_off,
               seg_bytes, group_bar(bars, i));
    }
  }
  for (int i = my_cnt + tid; i < stages; i += kThreads) mbar_arrive(group_bar(bars, i));

  const int tiles = (ncols + 15) >> 4;
  float acc[kMaxTilesPerWarp][4];
#pragma unroll
  for (int t = 0; t < kMaxTilesPerWarp; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;

  // H of the next group, prefetched: thread (k = tid / 8, s = tid % 8) for tid < 128
  const int hk = tid >> 3, hs = tid & 7;
  auto load_h = [&](int i) {                       // relu(sum of the K-slice partials)
    float v = 0.f;
    const size_t at = (size_t)(prt + i * P) * 8 + hs;
    for (int ks = 0; ks < a.ksplit; ++ks) v += a.H[(size_t)ks * a.h_stride + at];
    if (a.gate_mode == LIF_GATE_BUNDLED) {       // H = gate pre-activation, H2 = up value
      float u = 0.f;
      for (int ks = 0; ks < a.ksplit; ++ks) u += a.H2[(size_t)ks * a.h_stride + at];
      return apply_activation(v, a.act, a.act_thr) * u;
    }
    if (a.gate_mode == LIF_GATE_RESIDENT) {      // H = up value, gate from the score array
      if (hs >= a.S) return 0.f;
      const int id = a.pointers[max(0, row_slot(a, prt + i * P, base))];
      return apply_activation(a.gate_val[(size_t)hs * a.F + id], a.act, a.act_thr) * v;
    }
    return apply_activation(v, a.act, a.act_thr);
  };
  pdl_wait();                                      // H is complete from here on
  pdl_trigger();
  float h_next = 0.f;
  if (tid < 128 && hk < my_cnt) h_next = load_h(hk);
  // max |H| of a group is published one group ahead (after the MMAs, when the prefetched values
  // have landed), so that scaling costs no extra barrier
  auto publish_max = [&](int parity) {
    if (tid < 128) {
      float m = fabsf(h_next);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) gmax[parity][warp] = m;
    }
  };
  publish_max(0);
  __syncthreads();
  constexpr int kUnset = -1000;
  int h_exp = kUnset;              // H is scaled by 2^(10 - h_exp); kUnset: only zeros so far
  auto pow2 = [](int e) { return __int_as_float((127 + max(-126, min(127, e))) << 23); };

  int timed_out = 0;
  const int n_groups = (my_cnt + 15) >> 4;
  const int gq = lane >> 2, tq = lane & 3;
  for (int g = 0; g < n_groups; ++g) {
    const int st0 = (g & 1) * 16;
    const unsigned parity = (unsigned)(g >> 1) & 1u;
    const int valid = min(16, my_cnt - g * 16);
    {
      // the same for every thread: exponent of the largest |H| so far; accumulators follow
      const float m = fmaxf(fmaxf(gmax[g & 1][0], gmax[g & 1][1]), fmaxf(gmax[g & 1][2], gmax[g & 1][3]));
      if (m > 0.f && m < 3.0e38f) {
        const int e = (int)((__float_as_uint(m) >> 23) & 0xff) - 127;
        if (e > h_exp) {
          if (h_exp != kUnset) {
            const float f = pow2(h_exp - e);
#pragma unroll
            for (int t = 0; t < kMaxTilesPerWarp; ++t)
#pragma unroll
              for (int q = 0; q < 4; ++q) acc[t][q] *= f;
          }
          h_exp = e;
        }
      }
    }
    if (tid < 128) {
      const float h = (hk < valid ? h_next : 0.f) * (h_exp == kUnset ? 1.f : pow2(10 - h_exp));
      const __half hi = __float2half_rn(h);
      h_hi[hs * 16 + hk] = hi;
      h_lo[hs * 16 + hk] = __float2half_rn(h - __half2float(hi));
      const int i = (g + 1) * 16 + hk;
      h_next = i < my_cnt ? load_h(i) : 0.f;
    }
    if (!mbar_wait(bars + st0, parity, a.wait_polls)) timed_out = 1;
    if (__syncthreads_or(timed_out)) {
      if (tid == 0) {
        atomicCAS(a.status, LIF_OK, LIF_ERR_TIMEOUT);
        drain_ring(bars, stages, kGroup, g, stages / kGroup);
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
    publish_max((g + 1) & 1);                      // of the group just prefetched
    __syncthreads();                               // stages of this group and h_hi/h_lo are free
    if (tid < 16) {
      const int i = (g + 2) * 16 + tid;
      if (i < my_cnt) {
        const int slot = i < kRowCacheB ? slot_all[i] : max(0, row_slot(a, prt + i * P, base));
        mbar_expect_tx(bars + st0, seg_bytes);
        bulk_g2s(rows + (size_t)(st0 + tid) * pitch,
                 a.cache + (size_t)slot * a.row_elems + col_off, seg_bytes, bars + st0);
      } else {
        mbar_arrive(bars + st0);
      }
    }
  }
  // epilogue: acc[t] = (column gq (+8) of the tile, streams 2*tq, 2*tq + 1)
  float* out = a.y_partial + (size_t)prt * a.S * d;
  const float unscale = h_exp == kUnset ? 1.f : pow2(h_exp - 10);
#pragma unroll
  for (int t = 0; t < kMaxTilesPerWarp; ++t) {
    const int tile = warp + t * 8;
    if (tile < tiles) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int m = tile * 16 + gq + (e >> 1) * 8;
        const int s = tq * 2 + (e & 1);
        if (m < ncols && s < a.S) out[(size_t)s * d + col0 + m] = acc[t][e] * unscale;
      }
    }
  }
}

size_t up_smem(int k_per_split, int stages) {
  const size_t pitch = 2 * (size_t)k_per_split + kPad;
  return (8 + stages) * pitch + stages * 8 + stages * 4 + 8 * 32 * 4 * 4 + kRowCacheA * 8 + 16;
}
size_t down_smem(int cols_per_part, int stages) {
  return stages * (2 * (size_t)cols_per_part + kPad) + stages * 8 + 2 * 128 * 2 + kRowCacheB * 4 +
         2 * 4 * 4 + 16;
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
  const int tiles = d / 16;
  // phase A: split K over 1, 2, 4 or 8 CTAs until three 16-row groups fit beside the x slice
  int ksplit = 1, kps = d, st = 0;
  bool found = false;
  for (int want = 3 * kGroupA; want >= 2 * kGroupA && !found; want -= kGroupA)
    for (ksplit = 1; ksplit <= kBatchedMaxKSplit && !found; ksplit *= 2) {
      kps = (tiles + ksplit - 1) / ksplit * 16;
      st = want;
      found = up_smem(kps, st) <= (size_t)max_smem;
      if (found) break;
    }
  if (!found) return cudaSuccess;                  // fall back to the per-stream path
  // A CTA keeps only about 6-8 bulk copies in flight, so with short row slices two lighter
  // CTAs per SM (ring of two 8-row groups) move more bytes than one CTA with a deep ring.
  int up_group = kGroupA, up_ctas = 1;
  if (L->fb_up_two_ctas && ksplit > 1 && 2 * (up_smem(kps, 16) + 1024) <= (size_t)max_smem) {
    up_group = 8;
    up_ctas = 2;
    st = 16;
  }
  int parts = L->fb_parts_min > 0 ? L->fb_parts_min : 1;
  while ((tiles + parts - 1) / parts > 8 * kMaxTilesPerWarp ||
         down_smem((tiles + parts - 1) / parts * 16, 32) > (size_t)max_smem)
    ++parts;
  L->fb_ksplit = ksplit;
  L->fb_kps = kps;
  L->fb_up_group = up_group;
  L->fb_up_partitions = L->n_sm * up_ctas / ksplit > 0 ? L->n_sm * up_ctas / ksplit : 1;
  L->fb_up_stages = st;
  L->fb_up_smem = up_smem(kps, st);
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
  a.ksplit = L->fb_ksplit;
  a.k_per_split = L->fb_kps;
  a.up_partitions = L->fb_up_partitions;
  a.up_group = L->fb_up_group;
  a.h_stride = (size_t)D.d_ff * 8;
  a.act = D.activation;
  a.act_thr = D.activation_threshold;
  a.row_elems = row_elems(D);
  a.gate_mode = D.gate_mode;
  a.vec_off = 0;
  a.down_off = a.row_elems - D.d_model;
  a.add_bias = D.gate_mode != LIF_GATE_RESIDENT;   // resident gate: the bias is in the gate values
  a.F = D.d_ff;
  a.H2 = nullptr;
  a.gate_val = L->gate_val;
  a.pointers = L->pointers;
  a.rows = D.capacity;
  a.wait_polls = L->wait_polls;
  a.stages = L->fb_up_stages;
  cudaError_t e = launch_k(ffn_batched_up_kernel, dim3(L->fb_up_partitions * L->fb_ksplit),
                           dim3(kThreads), L->fb_up_smem, st, L->use_pdl, a);
  if (e != cudaSuccess) return e;
  if (D.gate_mode == LIF_GATE_BUNDLED) {           // second pass of phase A: the up rows
    float* h2 = L->h_rows + (size_t)kBatchedMaxKSplit * D.d_ff * 8;
    a.H = h2;
    a.vec_off = D.d_model;
    a.add_bias = 0;
    e = launch_k(ffn_batched_up_kernel, dim3(L->fb_up_partitions * L->fb_ksplit), dim3(kThreads),
                 L->fb_up_smem, st, L->use_pdl, a);
    if (e != cudaSuccess) return e;
    a.H = L->h_rows;
    a.H2 = h2;
  }
  a.stages = 32;
  e = launch_k(ffn_batched_down_kernel, dim3(L->fb_parts * L->fb_partitions), dim3(kThreads),
               L->fb_down_smem, st, L->use_pdl, a);
  if (e != cudaSuccess) return e;
  return launch_partial_sum(L, L->y_partial, n, L->fb_partitions, D.n_streams * D.d_model, y, st);
}

}  // namespace lif
