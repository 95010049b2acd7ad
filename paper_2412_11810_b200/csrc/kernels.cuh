// Device code of the BPTT step: spike compaction, event-driven forward step, surrogate-gradient
// backward step, sparse outer-product weight gradients, readout.  sm_100a, fp32.
//
// Arithmetic that decides spikes is written with explicit round-to-nearest intrinsics
// (__fadd_rn, __fmaf_rn, __fsub_rn, __fmul_rn) so that it is the same sequence of IEEE
// operations whatever the compiler flags: one accumulator per neuron, feed-forward events
// first, then recurrent events, each list in ascending presynaptic index, one fused
// multiply-add for the leak, one subtraction for the reset.
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tma.cuh"

namespace snnk {

namespace cg = cooperative_groups;

constexpr int MAXL = 8;
constexpr int FWD_THREADS = 128;            // each thread owns 4 adjacent neurons of one sample
constexpr int FWD_COLS = FWD_THREADS * 4;   // neurons per CTA
constexpr int LIST_CHUNK = 1024;            // events staged in shared memory at a time
constexpr int MAX_WORDS = 2048;             // 65536 neurons / 32
constexpr uint32_t STATUS_EVENT_OVERFLOW = 1u;
constexpr uint32_t STATUS_SYNC_TIMEOUT = 2u;     // a bounded wait (on a counter or an mbarrier) ran out
constexpr uint32_t STATUS_BAD_TARGET = 4u;   // a target outside [0, N_out)
constexpr uint32_t STATUS_DEBUG_CHECK = 8u;  // an index check of the bounds-checked build (SNN_DEBUG_CHECKS) failed

// Bounds-checked build (compiled with -DSNN_DEBUG_CHECKS=1): the data-dependent indices of the gather kernels -- a
// position in an event pool, the presynaptic row an event names -- are tested before use; a bad one raises
// STATUS_DEBUG_CHECK and is replaced by index 0, so that the access stays inside its array and the step ends with
// SNN_ERR_DEBUG_CHECK instead of a memory fault.  In the ordinary build the function is the identity.
__device__ __forceinline__ uint32_t checked_index(uint32_t idx, uint32_t limit, uint32_t* status) {
#ifdef SNN_DEBUG_CHECKS
  if (idx >= limit) {
    atomicOr(status, STATUS_DEBUG_CHECK);
    return 0u;
  }
#endif
  return idx;
}

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// 128-bit read-only load that does not allocate in L1: weight rows are streamed once per CTA.
__device__ __forceinline__ float4 ldg4_stream(const float* p) {
  float4 v;
  asm("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
      : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// 16-byte asynchronous copy global -> shared (bypasses L1 and the register file).  Copies are
// grouped with cp_async_commit; cp_async_wait<N> returns when at most N groups are pending.
// Each thread only ever reads back the bytes it copied itself, so no barrier is needed.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Programmatic dependent launch: every step kernel lets the next launch of the stream start early
// (its CTAs become resident and run their prologue while this grid drains) and waits for the
// previous grid to have completed, with its writes visible, before it touches global memory.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

constexpr uint32_t REC_TAG = 0x80000000u;  // list entry names a row of W_rec (else of W_ff)

// Valid bits of the last spike word of a row of n neurons.
__host__ __device__ __forceinline__ uint32_t last_word_mask(int n) {
  return (n & 31) ? (1u << (n & 31)) - 1u : 0xffffffffu;
}

// A row of spike words made of two parts that is addressed as one: the feed-forward source
// (layer below, this step) followed by the recurrent source (own layer, previous step).
struct WordPair {
  const uint32_t* a; int n_a;
  const uint32_t* b; int n_b;
  uint32_t a_last_mask = 0xffffffffu;   // valid bits of part a's last word (caller-owned input: its padding bits are ignored)
  __device__ __forceinline__ int size() const { return n_a + n_b; }
  __device__ __forceinline__ uint32_t get(int w) const {
    return w < n_a ? (w == n_a - 1 ? a[w] & a_last_mask : a[w]) : b[w - n_a];
  }
  __device__ __forceinline__ uint32_t first_index(int w) const {
    return w < n_a ? (uint32_t)w * 32u : ((uint32_t)(w - n_a) * 32u) | REC_TAG;
  }
};

// ------------------------------------------------------------------------------------------
// Spike compaction ("Spike Generation" in its sparse representation): spike words -> ascending
// index list.  Step 1: exclusive prefix sum of the per-word popcounts over the whole row.
// s_pref[w] = number of set bits in words [0, w), for w = 0 .. size() (the last one = total).
template <int NT>
__device__ uint32_t prefix_popcounts(const WordPair& wp, uint32_t* s_pref, uint32_t* s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_words = wp.size();
  const int wpt = (n_words + NT - 1) / NT;
  const int w0 = tid * wpt;
  uint32_t sum = 0;
  for (int i = 0; i < wpt; ++i)
    if (w0 + i < n_words) sum += __popc(wp.get(w0 + i));
  uint32_t inc = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += y;
  }
  __syncthreads();  // s_warp / s_pref may still be read from a previous use
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  uint32_t base = 0, total = 0;
#pragma unroll
  for (int k = 0; k < NT / 32; ++k) {
    uint32_t v = s_warp[k];
    if (k < warp) base += v;
    total += v;
  }
  uint32_t ex = base + inc - sum;
  for (int i = 0; i < wpt; ++i)
    if (w0 + i < n_words) { s_pref[w0 + i] = ex; ex += __popc(wp.get(w0 + i)); }
  if (tid == 0) s_pref[n_words] = total;
  __syncthreads();
  return total;
}

// Step 2a: the part [c0, c0 + LIST_CHUNK) of the list into shared memory.
template <int NT>
__device__ void fill_chunk_from_words(const WordPair& wp, const uint32_t* s_pref, uint32_t c0, uint32_t* s_list) {
  const int n_words = wp.size();
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = wp.get(w);
    if (!bits) continue;
    uint32_t p = s_pref[w];
    if (p >= c0 + LIST_CHUNK || p + __popc(bits) <= c0) continue;
    const uint32_t first = wp.first_index(w);
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p >= c0 && p < c0 + LIST_CHUNK) s_list[p - c0] = first + bit;
      ++p;
    }
  }
}

// Step 2a for the gather: instead of the indices, the address of each listed weight row (at the
// CTA's first column) goes to shared memory, so that issuing a row copy is one load and one add.
template <int NT>
__device__ void fill_rows_from_words(const WordPair& wp, const uint32_t* s_pref, uint32_t c0,
                                     const float* Wa_tile, const float* Wb_tile, int N, const float** s_row) {
  const int n_words = wp.size();
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = wp.get(w);
    if (!bits) continue;
    uint32_t p = s_pref[w];
    if (p >= c0 + LIST_CHUNK || p + __popc(bits) <= c0) continue;
    const bool in_a = w < wp.n_a;
    const float* base = (in_a ? Wa_tile : Wb_tile) + (size_t)((in_a ? w : w - wp.n_a) * 32) * N;
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p >= c0 && p < c0 + LIST_CHUNK) s_row[p - c0] = base + (size_t)bit * N;
      ++p;
    }
  }
}

// Step 2b: the lists to global memory (entries past the room left in a pool are dropped).
// Part a goes to dst_a (if not null), part b to dst_b; n_a_bits = set bits of part a.
// Graded events also store their value (read from the dense source rows val_a / val_b) and, per
// spike word, the number of events before it (pref_a / pref_b), which lets a reader find the
// position of a given neuron's event without searching.
template <int NT, bool GRADED>
__device__ void write_lists_from_words(const WordPair& wp, const uint32_t* s_pref, uint32_t n_a_bits,
                                       uint32_t* __restrict__ dst_a, uint32_t room_a,
                                       uint32_t* __restrict__ dst_b, uint32_t room_b,
                                       const float* __restrict__ val_a = nullptr, float* __restrict__ vdst_a = nullptr,
                                       uint16_t* __restrict__ pref_a = nullptr,
                                       const float* __restrict__ val_b = nullptr, float* __restrict__ vdst_b = nullptr,
                                       uint16_t* __restrict__ pref_b = nullptr) {
  const int n_words = wp.size();
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = wp.get(w);
    uint32_t p = s_pref[w];
    const bool in_a = w < wp.n_a;
    uint32_t* dst = in_a ? dst_a : dst_b;
    if (!dst) continue;
    const uint32_t room = in_a ? room_a : room_b;
    if (!in_a) p -= n_a_bits;
    const uint32_t first = wp.first_index(w) & ~REC_TAG;
    if (GRADED) (in_a ? pref_a : pref_b)[in_a ? w : w - wp.n_a] = (uint16_t)p;
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p < room) {
        dst[p] = first + bit;
        if (GRADED) (in_a ? vdst_a : vdst_b)[p] = (in_a ? val_a : val_b)[first + bit];
      }
      ++p;
    }
  }
}

// Step 2a for graded events: the values that go with fill_chunk_from_words' indices.
template <int NT>
__device__ void fill_values_from_words(const WordPair& wp, const uint32_t* s_pref, uint32_t c0,
                                       const float* __restrict__ val_a, const float* __restrict__ val_b,
                                       float* s_val) {
  const int n_words = wp.size();
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = wp.get(w);
    if (!bits) continue;
    uint32_t p = s_pref[w];
    if (p >= c0 + LIST_CHUNK || p + __popc(bits) <= c0) continue;
    const bool in_a = w < wp.n_a;
    const float* src = (in_a ? val_a : val_b) + (in_a ? w : w - wp.n_a) * 32;
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p >= c0 && p < c0 + LIST_CHUNK) s_val[p - c0] = src[bit];
      ++p;
    }
  }
}

// Dense fp32 rows -> spike words (bit = value is not zero): one warp per word.
__global__ void __launch_bounds__(256)
dense_to_words_kernel(const float* __restrict__ dense, size_t n_rows, int N, int W, uint32_t* __restrict__ words) {
  const size_t wid = ((size_t)blockIdx.x * 256 + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid >= n_rows * (size_t)W) return;
  const size_t row = wid / W;
  const int col = (int)(wid % W) * 32 + lane;
  const bool on = col < N && dense[row * N + col] != 0.f;
  const uint32_t m = __ballot_sync(0xffffffffu, on);
  if (lane == 0) words[wid] = m;
}

// Stand-alone compaction of many rows: one CTA per row.
__global__ void __launch_bounds__(FWD_THREADS)
compact_rows_kernel(const uint32_t* __restrict__ masks, int n_words, uint32_t* __restrict__ idx_out,
                    int capacity, uint32_t* __restrict__ count_out) {
  __shared__ uint32_t s_pref[MAX_WORDS + 1];
  __shared__ uint32_t s_warp[FWD_THREADS / 32];
  const size_t row = blockIdx.x;
  WordPair wp{masks + row * (size_t)n_words, n_words, nullptr, 0};
  const uint32_t total = prefix_popcounts<FWD_THREADS>(wp, s_pref, s_warp);
  write_lists_from_words<FWD_THREADS, false>(wp, s_pref, total, idx_out + row * (size_t)capacity,
                                             (uint32_t)capacity, nullptr, 0);
  if (threadIdx.x == 0) count_out[row] = total;
}

// ------------------------------------------------------------------------------------------
// Forward step (the paper's "MatMul" driven by sparse spikes, then "Spike Generation").
struct FwdLayer {
  const float* W_ff;          // [N_pre][N]
  const float* W_rec;         // [N][N]
  const float* V_prev;        // [B][N]  V_{t-1}
  float* V_out;               // [B][N]  V_t
  float* V_keep;              // optional second copy (checkpoint slot)
  float* V_dbg;               // optional third copy (inspection)
  const uint32_t* ff_mask;    // [B][W_pre] spikes of the layer below at step t      (generating mode)
  const uint32_t* rec_mask;   // [B][W]     own spikes at step t-1
  uint32_t* out_mask;         // [B][W]     own spikes at step t                      (generating mode)
  uint32_t* ff_pool;          // event pool of the layer below [B][ff_cap]
  uint32_t* ff_off;           // offsets row t of the layer below: [b] start, [B + b] end
  uint32_t* rec_pool;         // own event pool [B][rec_cap]
  uint32_t* rec_off;          // own offsets row t-1
  uint32_t* counts;           // [B][N] spike counts (last layer, generating mode) or null;
                              // the graded cell keeps the fp32 sum of its events there instead
  // graded cell only
  const float* ff_val_src;    // [B][N_pre] dense values of the layer below at step t   (generating mode)
  const float* rec_val_src;   // [B][N]     own dense event values at step t-1          (generating mode)
  float* act_out;             // [B][N]     own dense event values at step t            (generating mode)
  float* ff_vals;             // values that go with ff_pool
  float* rec_vals;            // values that go with rec_pool
  uint16_t* ff_pref;          // [B][W_pre] events before each spike word, layer below at step t
  uint16_t* rec_pref;         // [B][W]     the same for the own layer at step t-1
  uint32_t ff_cap, rec_cap;
  int N_pre, N, W_pre, W;
  int mode;                   // 0 idle, 1 step, 2 only write the list of own spikes at t-1
  int write_ff_list;          // the layer below is the input: this layer stores its lists
};

struct FwdParams {
  FwdLayer lay[MAXL];
  int B;
  float alpha, theta;
  uint32_t* status;
};

constexpr int GATHER_ROWS = 8;     // weight rows per copy group
constexpr int GATHER_STAGES = 3;   // groups of rows in the copy ring of a forward step (24 rows, 48 KB per CTA: three CTAs per SM)
constexpr size_t FWD_DYN_SMEM = (size_t)GATHER_STAGES * GATHER_ROWS * FWD_THREADS * sizeof(float4);

// The producer warp's share of a gather: the n listed rows (addresses in s_row) go into the ring as bulk copies, eight
// rows per group, up to four groups per trip round the loop (eight lanes each; one when the ring has few stages).
// `gc` counts the groups of the whole launch (the consumers count alike): group gc uses stage gc % G and the
// (gc / G)-th phase of its barriers.  A wait that runs out raises the status bit and sets `dead`.
__device__ __forceinline__ void gather_producer(const float* const* s_row, int n, unsigned char* ring, int G,
                                                uint64_t* s_full, uint64_t* s_empty, uint32_t row_bytes, int& gc, bool& dead,
                                                uint32_t* status, uint32_t group_bytes, uint32_t slot_row_bytes) {
  const int lane = threadIdx.x & 31, sub = lane >> 3, r = lane & 7;
  const int n_groups = (n + 7) / 8, NB = G >= 8 ? 4 : G >= 6 ? 2 : 1;   // a trip waits for all its stages: a fraction of the ring
  for (int g0 = 0; g0 < n_groups && !dead; g0 += NB) {
    const int g = g0 + sub;
    const bool valid = sub < NB && g < n_groups;
    const int my_gc = gc + sub, my_slot = my_gc % G;
    const uint32_t my_round = (uint32_t)(my_gc / G);
    bool ok = true;
    if (valid && my_gc >= G) ok = mbar_wait(s_empty + my_slot, (my_round - 1u) & 1u);   // group my_gc - G is added
    if (__any_sync(0xffffffffu, !ok)) {
      if (lane == 0) atomicOr(status, STATUS_SYNC_TIMEOUT);
      dead = true;
      break;
    }
    const int rows_here = valid ? (n - g * 8 < 8 ? n - g * 8 : 8) : 0;
    if (valid && r == 0) mbar_arrive_expect_tx(s_full + my_slot, (uint32_t)rows_here * row_bytes);
    __syncwarp();
    if (r < rows_here)
      bulk_load(ring + (size_t)my_slot * group_bytes + (size_t)r * slot_row_bytes, s_row[g * 8 + r], row_bytes, s_full + my_slot);
    gc += n_groups - g0 < NB ? n_groups - g0 : NB;
  }
}

// fwd_step_kernel: four consumer warps (a thread owns four neurons) and one producer warp.  The listed weight rows
// reach shared memory as plain bulk copies (`cp.async.bulk`, one row segment of this CTA's columns per copy, up to
// 2 KB), eight rows per group, issued by eight lanes of the producer warp at once; groups cycle through a ring of
// GATHER_STAGES stages guarded by full / empty mbarriers.  The consumers issue no copies: per row and thread one
// 16-byte shared-memory read and four additions, in list order.
constexpr int FWDS_THREADS = FWD_THREADS + 32;
constexpr uint32_t FWDS_ROW_BYTES = FWD_COLS * sizeof(float);                  // a row segment in the ring
constexpr uint32_t FWDS_GROUP_BYTES = GATHER_ROWS * FWDS_ROW_BYTES;

template <bool GEN, bool GRADED>
__global__ void __launch_bounds__(FWDS_THREADS) fwd_step_kernel(const __grid_constant__ FwdParams p) {
  pdl_launch_dependents();
  const FwdLayer& L = p.lay[blockIdx.z];
  if (L.mode == 0) return;
  const int col0 = blockIdx.x * FWD_COLS;
  if (col0 >= L.N) return;
  const int b = blockIdx.y, B = p.B;
  const bool tile0 = blockIdx.x == 0;
  __shared__ const float* s_row[LIST_CHUNK];   // addresses of the listed weight rows at this CTA's first column
  __shared__ uint32_t s_pref[GEN ? 2 * MAX_WORDS + 1 : 1];
  __shared__ uint32_t s_warp[FWDS_THREADS / 32];
  __shared__ float s_val[GRADED ? LIST_CHUNK : 1];
  __shared__ uint64_t s_full[GATHER_STAGES], s_empty[GATHER_STAGES];
  extern __shared__ float4 s_stage[];   // [GATHER_STAGES][GATHER_ROWS][FWD_THREADS]
  const bool producer = threadIdx.x >= FWD_THREADS;        // the fifth warp
  const int col = col0 + threadIdx.x * 4;
  const bool active = !producer && col < L.N;
  const bool step = L.mode == 1;
  if (!step && !(GEN && tile0)) return;
  if (threadIdx.x == 0) {
    for (int i = 0; i < GATHER_STAGES; ++i) { mbar_init(s_full + i, 1); mbar_init(s_empty + i, FWD_THREADS / 32); }
    mbar_fence_init();
  }
  __syncthreads();

  pdl_wait();
  // issue the loads the epilogue needs before anything else
  float4 vp = make_float4(0.f, 0.f, 0.f, 0.f);
  uint32_t pw = 0;
  if (step && active) {
    vp = *reinterpret_cast<const float4*>(L.V_prev + (size_t)b * L.N + col);
    if (!GRADED) pw = L.rec_mask[(size_t)b * L.W + (col >> 5)] >> (col & 31);
  }

  // ---- the two event lists of this step as one: feed-forward events, then recurrent events
  uint32_t n_ff, total, s_ff = 0, s_rec = 0;
  uint32_t* const ff_pool = L.ff_pool + (size_t)b * L.ff_cap;
  uint32_t* const rec_pool = L.rec_pool + (size_t)b * L.rec_cap;
  WordPair wp{nullptr, 0, nullptr, 0};
  if (GEN) {
    wp = WordPair{step ? L.ff_mask + (size_t)b * L.W_pre : nullptr, step ? L.W_pre : 0,
                  L.rec_mask + (size_t)b * L.W, L.W, last_word_mask(L.N_pre)};
    total = prefix_popcounts<FWDS_THREADS>(wp, s_pref, s_warp);
    n_ff = s_pref[wp.n_a];
    if (tile0) {  // this CTA appends the lists to the event pools
      const bool wr_ff = step && L.write_ff_list;
      s_rec = L.rec_off[b];
      if (wr_ff) s_ff = L.ff_off[b];
      const uint32_t room_ff = wr_ff ? L.ff_cap - s_ff : 0, room_rec = L.rec_cap - s_rec;
      if (GRADED)
        write_lists_from_words<FWDS_THREADS, true>(
            wp, s_pref, n_ff, wr_ff ? ff_pool + s_ff : nullptr, room_ff, rec_pool + s_rec, room_rec,
            wr_ff ? L.ff_val_src + (size_t)b * L.N_pre : nullptr, L.ff_vals + (size_t)b * L.ff_cap + s_ff,
            L.ff_pref + (size_t)b * L.W_pre, L.rec_val_src + (size_t)b * L.N,
            L.rec_vals + (size_t)b * L.rec_cap + s_rec, L.rec_pref + (size_t)b * L.W);
      else
        write_lists_from_words<FWDS_THREADS, false>(wp, s_pref, n_ff, wr_ff ? ff_pool + s_ff : nullptr, room_ff,
                                                   rec_pool + s_rec, room_rec);
      if (threadIdx.x == 0) {
        const uint32_t n_rec = total - n_ff;
        L.rec_off[B + b] = s_rec + (n_rec < room_rec ? n_rec : room_rec);
        if (wr_ff) L.ff_off[B + b] = s_ff + (n_ff < room_ff ? n_ff : room_ff);
        if (n_rec > room_rec || (wr_ff && n_ff > room_ff)) atomicOr(p.status, STATUS_EVENT_OVERFLOW);
      }
    }
    if (!step) return;
  } else {
    s_ff = L.ff_off[b]; n_ff = L.ff_off[B + b] - s_ff;
    s_rec = L.rec_off[b]; total = n_ff + (L.rec_off[B + b] - s_rec);
  }

  // ---- gather-accumulate in list order
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // ring position of the next group (both roles count the groups of all chunks alike); bytes of a row segment
  int gc = 0, slot = 0;
  uint32_t round = 0;          // gc / GATHER_STAGES
  bool dead = false;           // a wait of this warp ran out: no more waiting, copying or adding
  const uint32_t row_bytes = (uint32_t)(L.N - col0 < FWD_COLS ? L.N - col0 : FWD_COLS) * sizeof(float);
  const float* const Wff_tile = L.W_ff + col0;
  const float* const Wrec_tile = L.W_rec + col0;
  for (uint32_t c0 = 0; c0 < total; c0 += LIST_CHUNK) {
    const int n = (int)(total - c0 < (uint32_t)LIST_CHUNK ? total - c0 : (uint32_t)LIST_CHUNK);
    if (GEN) {
      fill_rows_from_words<FWDS_THREADS>(wp, s_pref, c0, Wff_tile, Wrec_tile, L.N, s_row);
      if (GRADED)
        fill_values_from_words<FWDS_THREADS>(wp, s_pref, c0, L.ff_val_src + (size_t)b * L.N_pre,
                                            L.rec_val_src + (size_t)b * L.N, s_val);
    } else {
      for (int i = threadIdx.x; i < n; i += FWDS_THREADS) {
        const uint32_t q = c0 + i;
        s_row[i] = q < n_ff
            ? Wff_tile + (size_t)checked_index(ff_pool[checked_index(s_ff + q, L.ff_cap, p.status)], L.N_pre, p.status) * L.N
            : Wrec_tile + (size_t)checked_index(rec_pool[checked_index(s_rec + (q - n_ff), L.rec_cap, p.status)], L.N, p.status) * L.N;
        if (GRADED)
          s_val[i] = q < n_ff ? L.ff_vals[(size_t)b * L.ff_cap + s_ff + q]
                              : L.rec_vals[(size_t)b * L.rec_cap + s_rec + (q - n_ff)];
      }
    }
    __syncthreads();
    const int n_groups = (n + GATHER_ROWS - 1) / GATHER_ROWS;
    if (producer) {
      // ---- producer warp: eight lanes copy the eight rows of a group (the loop holds nothing else: with three stages
      // its trips bound the gather, and the general routine above, four groups per trip, is slower here)
      const int lane = threadIdx.x & 31;
      for (int g = 0; g < n_groups && !dead; ++g) {
        if (gc >= GATHER_STAGES && !mbar_wait(s_empty + slot, (round - 1u) & 1u)) {   // group gc - GATHER_STAGES is added
          if (lane == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          dead = true;
          break;
        }
        const int rows_here = n - g * GATHER_ROWS < GATHER_ROWS ? n - g * GATHER_ROWS : GATHER_ROWS;
        if (lane == 0) mbar_arrive_expect_tx(s_full + slot, (uint32_t)rows_here * row_bytes);
        __syncwarp();
        if (lane < rows_here)
          bulk_load(reinterpret_cast<unsigned char*>(s_stage) + (size_t)slot * FWDS_GROUP_BYTES + (size_t)lane * FWDS_ROW_BYTES,
                    s_row[g * GATHER_ROWS + lane], row_bytes, s_full + slot);
        ++gc;
        if (++slot == GATHER_STAGES) { slot = 0; ++round; }
      }
    } else {
      // ---- consumers: the rows of a group in list order
      auto add_row = [&](const float4 w, int i) {
        if (GRADED) {   // one fused multiply-add per event and neuron
          const float sv = s_val[i];
          acc.x = __fmaf_rn(sv, w.x, acc.x); acc.y = __fmaf_rn(sv, w.y, acc.y);
          acc.z = __fmaf_rn(sv, w.z, acc.z); acc.w = __fmaf_rn(sv, w.w, acc.w);
        } else {        // a binary spike: the fused multiply-add is an exact plain add
          acc.x = __fadd_rn(acc.x, w.x); acc.y = __fadd_rn(acc.y, w.y);
          acc.z = __fadd_rn(acc.z, w.z); acc.w = __fadd_rn(acc.w, w.w);
        }
      };
      for (int g = 0; g < n_groups && !dead; ++g) {
        if (!mbar_wait(s_full + slot, round & 1u)) {
          if ((threadIdx.x & 31) == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          dead = true;
          break;
        }
        if (active) {
          const float4* src = s_stage + (size_t)slot * GATHER_ROWS * FWD_THREADS + threadIdx.x;
          if ((g + 1) * GATHER_ROWS <= n) {
#pragma unroll
            for (int u = 0; u < GATHER_ROWS; ++u) add_row(src[u * FWD_THREADS], g * GATHER_ROWS + u);
          } else {
#pragma unroll
            for (int u = 0; u < GATHER_ROWS; ++u)
              if (g * GATHER_ROWS + u < n) add_row(src[u * FWD_THREADS], g * GATHER_ROWS + u);
          }
        }
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(s_empty + slot);
        ++gc;
        if (++slot == GATHER_STAGES) { slot = 0; ++round; }
      }
    }
    __syncthreads();
  }
  if (producer) {
    if (dead)   // the copies of the last groups issued may still be on their way: wait for them, briefly
      for (int cc = gc > GATHER_STAGES ? gc - GATHER_STAGES : 0; cc < gc; ++cc)
        mbar_wait(s_full + cc % GATHER_STAGES, (uint32_t)(cc / GATHER_STAGES) & 1u, 1u << 14);
    return;
  }

  // ---- leak, reset by subtraction of the previous step's own spike, threshold
  uint32_t nib = 0;
  if (active) {
    const size_t k = (size_t)b * L.N + col;
    float4 v;
    if (GRADED) {   // leaky integrator without reset
      v.x = __fmaf_rn(p.alpha, vp.x, acc.x); v.y = __fmaf_rn(p.alpha, vp.y, acc.y);
      v.z = __fmaf_rn(p.alpha, vp.z, acc.z); v.w = __fmaf_rn(p.alpha, vp.w, acc.w);
    } else {
      v.x = __fsub_rn(__fmaf_rn(p.alpha, vp.x, acc.x), __fmul_rn(p.theta, (float)(pw & 1u)));
      v.y = __fsub_rn(__fmaf_rn(p.alpha, vp.y, acc.y), __fmul_rn(p.theta, (float)((pw >> 1) & 1u)));
      v.z = __fsub_rn(__fmaf_rn(p.alpha, vp.z, acc.z), __fmul_rn(p.theta, (float)((pw >> 2) & 1u)));
      v.w = __fsub_rn(__fmaf_rn(p.alpha, vp.w, acc.w), __fmul_rn(p.theta, (float)((pw >> 3) & 1u)));
    }
    *reinterpret_cast<float4*>(L.V_out + k) = v;
    if (L.V_keep) *reinterpret_cast<float4*>(L.V_keep + k) = v;
    if (L.V_dbg) *reinterpret_cast<float4*>(L.V_dbg + k) = v;
    if (GEN) {
      nib = (v.x > p.theta ? 1u : 0u) | (v.y > p.theta ? 2u : 0u) | (v.z > p.theta ? 4u : 0u) |
            (v.w > p.theta ? 8u : 0u);
      if (GRADED) {
        const float4 a = make_float4(nib & 1u ? v.x : 0.f, nib & 2u ? v.y : 0.f, nib & 4u ? v.z : 0.f,
                                     nib & 8u ? v.w : 0.f);
        *reinterpret_cast<float4*>(L.act_out + k) = a;
        if (L.counts && nib) {   // time-summed events, added in step order
          float4* c = reinterpret_cast<float4*>(L.counts + k);
          float4 cv = *c;
          cv.x = __fadd_rn(cv.x, a.x); cv.y = __fadd_rn(cv.y, a.y);
          cv.z = __fadd_rn(cv.z, a.z); cv.w = __fadd_rn(cv.w, a.w);
          *c = cv;
        }
      } else if (L.counts && nib) {
        uint4* c = reinterpret_cast<uint4*>(L.counts + k);
        uint4 cv = *c;
        cv.x += nib & 1u; cv.y += (nib >> 1) & 1u; cv.z += (nib >> 2) & 1u; cv.w += (nib >> 3) & 1u;
        *c = cv;
      }
    }
  }
  if (GEN) {
    // eight neighbouring lanes hold the 32 bits of one spike word
    const int lane = threadIdx.x & 31;
    uint32_t word = nib << (4 * (lane & 7));
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    word |= __shfl_xor_sync(0xffffffffu, word, 4);
    const int widx = col >> 5;
    if ((lane & 7) == 0 && widx < L.W) L.out_mask[(size_t)b * L.W + widx] = word;
  }
}

// 16-byte asynchronous copy, or 16 zero bytes when `real` is false (nothing is read then).
__device__ __forceinline__ void cp_async16_or_zero(void* smem_dst, const void* gmem_src, bool real) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(gmem_src), "r"(real ? 16u : 0u) : "memory");
}

// L2 eviction priorities for copies that name one: lines fetched with `l2_keep_policy` are the last to be evicted,
// lines fetched with `l2_stream_policy` the first.
__device__ __forceinline__ uint64_t l2_keep_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_stream_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// ------------------------------------------------------------------------------------------
// Re-forward of a run of steps in two launches (the recomputation passes of Sec. 3).
//
// Once the forward pass has stored the events of every step, the input current
// I_t = S^{l-1}_t W_ff + S^l_{t-1} W_rec of any step can be computed without the steps before it:
// only the leak/reset recurrence V_t = alpha V_{t-1} + I_t - theta S_{t-1} is sequential, and it is
// elementwise.  refwd_gather_kernel computes I_t for all steps of the run at once (one CTA per
// step, sample, layer and column tile: enough warps per SM to keep the L2 gather busy) and leaves
// it where V_t will go; refwd_scan_kernel then walks through the steps and replaces I_t by V_t.
// Per neuron the arithmetic is that of fwd_step_kernel, operation for operation.
struct SegLayer {
  const float* W_ff;          // [N_pre][N]
  const float* W_rec;         // [N][N]
  const uint32_t* ff_pool;    // event pool of the layer below [B][ff_cap]
  const uint32_t* ff_off;     // its offsets, row 0: list (t, b) = [off[t * B + b], off[(t + 1) * B + b])
  const uint32_t* rec_pool;   // own event pool [B][rec_cap]
  const uint32_t* rec_off;    // own offsets, row 0
  const float* ff_vals;       // graded cell: values that go with ff_pool
  const float* rec_vals;      // graded cell: values that go with rec_pool
  size_t state_off;           // offset of this layer inside a state slot, in floats
  uint32_t ff_cap, rec_cap;
  int N, N_pre;
};

struct SegParams {
  SegLayer lay[MAXL];
  uint32_t* status;
  float* slots;               // state slot s starts at slots + s * slot_stride
  size_t slot_stride;         // floats
  int B;
  int t0;                     // the operation computes steps t0+1 .. from the state of step t0
  int d0, n;                  // this run: steps t0+d0+1 .. t0+d0+n
  int buf_slot, buf_len;      // step t0+d goes to slot buf_slot + (d-1) % buf_len (as in snn_op)
  int tiles;                  // refwd_gather_kernel: column tiles of the widest layer
};

constexpr int RG_ROWS = 4;     // weight rows per copy group
constexpr int RG_STAGES = 5;   // copy groups in flight per thread (20 rows, 40 KB per CTA: four CTAs per SM)
constexpr size_t REFWD_DYN_SMEM = (size_t)RG_STAGES * RG_ROWS * FWD_THREADS * sizeof(float4);

template <bool GRADED>
__global__ void __launch_bounds__(FWD_THREADS, 4) refwd_gather_kernel(const __grid_constant__ SegParams p) {
  pdl_launch_dependents();
  // grid (sample, step, layer x column tile): the thread blocks that run together work on the same 512 columns
  // of one layer, so whatever the size of the network the rows they gather stay in L2 between them
  const int l = blockIdx.z / p.tiles, d = p.d0 + 1 + blockIdx.y;
  const SegLayer& L = p.lay[l];
  const int col0 = (blockIdx.z % p.tiles) * FWD_COLS;
  if (col0 >= L.N) return;
  const int b = blockIdx.x, B = p.B, tid = threadIdx.x, t = p.t0 + d;
  __shared__ const float* s_row[LIST_CHUNK];
  __shared__ float s_val[GRADED ? LIST_CHUNK : 1];
  extern __shared__ float4 s_stage[];   // [RG_STAGES][RG_ROWS][FWD_THREADS]
  const int col = col0 + tid * 4;
  const bool active = col < L.N;
  const float* const Wff_tile = L.W_ff + col0;
  const float* const Wrec_tile = L.W_rec + col0;
  const uint32_t* const ff_pool = L.ff_pool + (size_t)b * L.ff_cap;
  const uint32_t* const rec_pool = L.rec_pool + (size_t)b * L.rec_cap;

  pdl_wait();
  const uint32_t s_ff = L.ff_off[(size_t)t * B + b], n_ff = L.ff_off[(size_t)(t + 1) * B + b] - s_ff;
  const uint32_t s_rec = L.rec_off[(size_t)(t - 1) * B + b], total = n_ff + (L.rec_off[(size_t)t * B + b] - s_rec);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (uint32_t c0 = 0; c0 < total; c0 += LIST_CHUNK) {
    const int n = (int)(total - c0 < (uint32_t)LIST_CHUNK ? total - c0 : (uint32_t)LIST_CHUNK);
    for (int i = tid; i < n; i += FWD_THREADS) {
      const uint32_t q = c0 + i;
      s_row[i] = q < n_ff
          ? Wff_tile + (size_t)checked_index(ff_pool[checked_index(s_ff + q, L.ff_cap, p.status)], L.N_pre, p.status) * L.N
          : Wrec_tile + (size_t)checked_index(rec_pool[checked_index(s_rec + (q - n_ff), L.rec_cap, p.status)], L.N, p.status) * L.N;
      if (GRADED)
        s_val[i] = q < n_ff ? L.ff_vals[(size_t)b * L.ff_cap + s_ff + q]
                            : L.rec_vals[(size_t)b * L.rec_cap + s_rec + (q - n_ff)];
    }
    __syncthreads();
    if (active) {
      float4* const ring = s_stage + tid;
      const int n_groups = (n + RG_ROWS - 1) / RG_ROWS;
      const int lane_col = tid * 4;
      auto issue = [&](int g) {
        if (g < n_groups) {
          float4* dst = ring + (size_t)(g % RG_STAGES) * RG_ROWS * FWD_THREADS;
          const float* const* rows = s_row + g * RG_ROWS;
#pragma unroll
          for (int u = 0; u < RG_ROWS; ++u) {   // past the list's end: a zero-filled copy (+0 leaves the sum unchanged)
            const bool real = g * RG_ROWS + u < n;
            cp_async16_or_zero(dst + u * FWD_THREADS, real ? rows[u] + lane_col : Wff_tile, real);
          }
        }
        cp_async_commit();
      };
      for (int g = 0; g < RG_STAGES - 1; ++g) issue(g);
      for (int g = 0; g < n_groups; ++g) {
        issue(g + RG_STAGES - 1);
        cp_async_wait<RG_STAGES - 1>();
        const float4* src = ring + (size_t)(g % RG_STAGES) * RG_ROWS * FWD_THREADS;
#pragma unroll
        for (int u = 0; u < RG_ROWS; ++u) {
          const float4 w = src[u * FWD_THREADS];
          if (GRADED) {
            const int i = g * RG_ROWS + u;
            const float sv = i < n ? s_val[i] : 0.f;
            acc.x = __fmaf_rn(sv, w.x, acc.x); acc.y = __fmaf_rn(sv, w.y, acc.y);
            acc.z = __fmaf_rn(sv, w.z, acc.z); acc.w = __fmaf_rn(sv, w.w, acc.w);
          } else {
            acc.x = __fadd_rn(acc.x, w.x); acc.y = __fadd_rn(acc.y, w.y);
            acc.z = __fadd_rn(acc.z, w.z); acc.w = __fadd_rn(acc.w, w.w);
          }
        }
      }
      cp_async_wait<0>();
    }
    __syncthreads();
  }
  if (active)
    *reinterpret_cast<float4*>(p.slots + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride + L.state_off +
                               (size_t)b * L.N + col) = acc;
}

// The recurrence over the steps of a run.  A state slot is one flat array (all layers, [B][N_l] each) and
// the update is elementwise, so a thread owns four adjacent floats of it and needs no layer arithmetic.
struct ScanParams {
  float* slots;
  size_t slot_stride;         // floats
  size_t n_quads;             // float4 per state
  const float* v_start;       // state of step t0+d0 (a slot, or `carry` of the previous run)
  float* carry;               // receives the state of the run's last step
  int t0, d0, n;
  int buf_slot, buf_len, keep_every, keep_slot;
  float alpha, theta;
};

constexpr int SCAN_BATCH = 8;   // steps whose loads are in flight together

template <bool GRADED>
__global__ void __launch_bounds__(128) refwd_scan_kernel(const __grid_constant__ ScanParams p) {
  pdl_launch_dependents();
  const size_t q = (size_t)blockIdx.x * 128 + threadIdx.x;
  if (q >= p.n_quads) return;
  pdl_wait();
  float4 v = reinterpret_cast<const float4*>(p.v_start)[q];
  // spikes of the previous step: S_0 = 0, later S_t = [V_t > theta]
  uint32_t sp = 0;
  if (!GRADED && p.t0 + p.d0 > 0)
    sp = (v.x > p.theta ? 1u : 0u) | (v.y > p.theta ? 2u : 0u) | (v.z > p.theta ? 4u : 0u) | (v.w > p.theta ? 8u : 0u);
  for (int i0 = 0; i0 < p.n; i0 += SCAN_BATCH) {
    float4 I[SCAN_BATCH];
    float4* where[SCAN_BATCH];
#pragma unroll
    for (int u = 0; u < SCAN_BATCH; ++u) {
      const int d = p.d0 + i0 + u + 1;
      where[u] = reinterpret_cast<float4*>(p.slots + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride) + q;
      I[u] = i0 + u < p.n ? *where[u] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < SCAN_BATCH; ++u) {
      if (i0 + u < p.n) {
        if (GRADED) {
          v.x = __fmaf_rn(p.alpha, v.x, I[u].x); v.y = __fmaf_rn(p.alpha, v.y, I[u].y);
          v.z = __fmaf_rn(p.alpha, v.z, I[u].z); v.w = __fmaf_rn(p.alpha, v.w, I[u].w);
        } else {
          v.x = __fsub_rn(__fmaf_rn(p.alpha, v.x, I[u].x), __fmul_rn(p.theta, (float)(sp & 1u)));
          v.y = __fsub_rn(__fmaf_rn(p.alpha, v.y, I[u].y), __fmul_rn(p.theta, (float)((sp >> 1) & 1u)));
          v.z = __fsub_rn(__fmaf_rn(p.alpha, v.z, I[u].z), __fmul_rn(p.theta, (float)((sp >> 2) & 1u)));
          v.w = __fsub_rn(__fmaf_rn(p.alpha, v.w, I[u].w), __fmul_rn(p.theta, (float)((sp >> 3) & 1u)));
          sp = (v.x > p.theta ? 1u : 0u) | (v.y > p.theta ? 2u : 0u) | (v.z > p.theta ? 4u : 0u) |
               (v.w > p.theta ? 8u : 0u);
        }
        *where[u] = v;
        const int d = p.d0 + i0 + u + 1;
        if (p.keep_every > 0 && d % p.keep_every == 0)
          reinterpret_cast<float4*>(p.slots + (size_t)(p.keep_slot + d / p.keep_every - 1) * p.slot_stride)[q] = v;
      }
    }
  }
  reinterpret_cast<float4*>(p.carry)[q] = v;
}

// ------------------------------------------------------------------------------------------
// Input currents of a run of steps with the weight rows as the stationary operand (recomputation passes
// of networks whose weights do not stay in L2).
//
// The gather above reads, for every (step, sample), each active weight row again: 16 steps x 8 samples at
// 5 % activity touch every row about six times.  Here a CTA owns a slab of RR_COLS columns and a block of
// (step, sample) pairs of the run, walks through the presynaptic rows in ascending order (feed-forward rows,
// then recurrent ones), reads each row ONCE, and adds it to the accumulators of exactly those pairs in which
// that neuron fired.  Per accumulator this is the sequence of additions of fwd_step_kernel (feed-forward
// events ascending, then recurrent events ascending, starting from zero), hence the same bits.
//
// Two launches.  rows_events_kernel turns the stored spike words of the run into two 32-bit words per
// (block of 32 rows, pair): the number of firing rows of that block, and up to four row numbers, one per byte
// (a block with more keeps its raw spike word instead).  refwd_rows_kernel then streams the rows: one
// elected thread issues, per block of 32 rows, one tiled bulk copy (TMA) of the [32 rows][128 columns] tile
// and one bulk copy of the pairs' event words into a ring of RR_STAGES stages guarded by full / empty
// mbarriers; the other warps consume: a warp owns 4 pairs, a lane four adjacent columns (4 float4
// accumulators per thread, named statically), and an event is one 16-byte shared-memory read and two packed
// fp32 additions.
struct RowsLayer {
  const uint32_t* ff_words;   // spike words of the layer below; row of step t at (t - ff_row0) * B * W_pre
  const uint32_t* words;      // own spike words [T+1][B][W]
  size_t state_off;           // offset of this layer inside a state slot, in floats
  size_t ev_off;              // this layer's event words inside `events`, in words: [W_pre + W][ev_stride]
  int N_pre, N, W_pre, W;
  int ff_row0;                // 1 for the input (its rows start at step 1), 0 for hidden layers
};

struct RowsParams {
  CUtensorMap map_ff[MAXL];   // W_ff^l [N_pre][N], box 32 rows x 128 columns
  CUtensorMap map_rec[MAXL];  // W_rec^l [N][N]
  RowsLayer lay[MAXL];
  float* slots;               // state slot s starts at slots + s * slot_stride
  size_t slot_stride;         // floats
  uint32_t* events;           // event counts of the run; the row-number words follow at + raw_off
  size_t raw_off;             // words
  uint32_t* status;
  int ev_stride;              // pairs rounded up to whole CTA blocks
  int B;
  int t0;                     // the operation computes steps t0+1 .. from the state of step t0
  int d0, n;                  // this run: steps t0+d0+1 .. t0+d0+n
  int buf_slot, buf_len;      // step t0+d goes to slot buf_slot + (d-1) % buf_len (as in snn_op)
  int pb;                     // (step, sample) pairs per CTA: 16, 32, 64 or 128, one consumer warp per 8
};

constexpr int RR_COLS = 128;     // columns per CTA (32 lanes x 4)
constexpr int RR_ROWS = 32;      // rows per tile: one spike word
constexpr int RR_STAGES = 4;     // tiles in flight per CTA
constexpr int RR_PPW = 4;        // pairs per consumer warp (16 accumulator registers per thread: many warps per SM
                                 // hide the shared-memory latency of the data-dependent row reads; eight pairs per
                                 // warp, half the warps: 69 against 60 ms for a pass over the largest benchmark network)
constexpr int RR_MAX_PB = 64;    // at most 16 consumer warps
constexpr uint32_t RR_TILE_BYTES = RR_ROWS * RR_COLS * sizeof(float);
constexpr uint32_t RR_STAGE_BYTES = RR_TILE_BYTES + RR_COLS * sizeof(float);   // the tile and one row of zeros after it
constexpr uint32_t RR_EV_MANY = 7u;   // count field of an event word whose block has more than four firing rows
__host__ __device__ inline size_t refwd_rows_smem_bytes(int pb) {
  return (size_t)RR_STAGES * (RR_STAGE_BYTES + 2 * (size_t)pb * sizeof(uint32_t)) + 2 * RR_STAGES * sizeof(uint64_t);
}

// Event words of the run: thread = (pair, block of 32 rows, layer).
__global__ void __launch_bounds__(128) rows_events_kernel(const __grid_constant__ RowsParams p) {
  pdl_launch_dependents();
  const RowsLayer& L = p.lay[blockIdx.z];
  const int rb = blockIdx.y, pair = blockIdx.x * 128 + threadIdx.x;
  if (rb >= L.W_pre + L.W || pair >= p.ev_stride) return;
  pdl_wait();
  uint32_t bits = 0;
  if (pair < p.n * p.B) {
    const int t = p.t0 + p.d0 + 1 + pair / p.B, b = pair % p.B;
    if (rb < L.W_pre) {
      bits = L.ff_words[((size_t)(t - L.ff_row0) * p.B + b) * L.W_pre + rb];
      if (rb == L.W_pre - 1) bits &= last_word_mask(L.N_pre);   // the input's padding bits are ignored
    } else {
      bits = L.words[((size_t)(t - 1) * p.B + b) * L.W + (rb - L.W_pre)];
    }
  }
  // first word: the number of firing rows (RR_EV_MANY if more than four) and, in bytes 1 and 2, the first two of
  // them; second word: the third and fourth in bytes 0 and 1 -- or the raw spike word when there are more than four.
  // A row that does not exist is written as RR_ROWS: the consumer's tile has one more row, of zeros, so that it can
  // add the first row of every pair without looking at the count (x + 0 = x exactly, and no accumulator is ever -0)
  const uint32_t cnt = __popc(bits);
  uint32_t r[4] = {RR_ROWS, RR_ROWS, RR_ROWS, RR_ROWS};
  {
    uint32_t rest = bits;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (rest) {
        r[k] = (uint32_t)(__ffs(rest) - 1);
        rest &= rest - 1;
      }
    }
  }
  const uint32_t w = (cnt <= 4 ? cnt : RR_EV_MANY) | r[0] << 8 | r[1] << 16;
  const uint32_t rows = cnt <= 4 ? (r[2] | r[3] << 8) : bits;
  const size_t at = L.ev_off + (size_t)rb * p.ev_stride + pair;
  p.events[at] = w;
  p.events[p.raw_off + at] = rows;
}

__device__ __forceinline__ void lds_2x64(uint32_t saddr, unsigned long long& a, unsigned long long& b) {
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(saddr));
}
// two fp32 lanes per register pair: a += w, each element rounded to nearest even (as __fadd_rn)
__device__ __forceinline__ void add_f32x2(unsigned long long& a, const unsigned long long w) {
  asm("add.rn.f32x2 %0, %0, %1;" : "+l"(a) : "l"(w));
}

__global__ void __launch_bounds__(32 * (RR_MAX_PB / RR_PPW + 1)) refwd_rows_kernel(const __grid_constant__ RowsParams p) {
  pdl_launch_dependents();
  const int l = blockIdx.z;
  const RowsLayer& L = p.lay[l];
  const int col0 = blockIdx.y * RR_COLS;
  const int pairs = p.n * p.B, pair0 = blockIdx.x * p.pb;
  if (col0 >= L.N || pair0 >= pairs) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_consumers = p.pb / RR_PPW;            // consumer warps 0 .. n_consumers-1, then the producer warp
  extern __shared__ __align__(128) unsigned char s_raw_bytes[];
  unsigned char* const s_tiles = s_raw_bytes;                                 // [RR_STAGES]: [32][128] fp32, then 128 zeros
  uint32_t* const s_ev = reinterpret_cast<uint32_t*>(s_raw_bytes + (size_t)RR_STAGES * RR_STAGE_BYTES);   // [RR_STAGES][2][pb]
  uint64_t* const s_full = reinterpret_cast<uint64_t*>(s_ev + (size_t)RR_STAGES * 2 * p.pb);       // [RR_STAGES]
  uint64_t* const s_empty = s_full + RR_STAGES;
  const int n_blocks = L.W_pre + L.W;
  if (tid == 0) {
    for (int s = 0; s < RR_STAGES; ++s) { mbar_init(s_full + s, 1); mbar_init(s_empty + s, n_consumers); }
    mbar_fence_init();
  }
  for (int q = tid; q < RR_STAGES * RR_COLS; q += blockDim.x)   // the row of zeros behind every tile
    reinterpret_cast<float*>(s_tiles + (size_t)(q / RR_COLS) * RR_STAGE_BYTES + RR_TILE_BYTES)[q % RR_COLS] = 0.f;
  __syncthreads();
  pdl_wait();
  const uint32_t ev_bytes = (uint32_t)p.pb * sizeof(uint32_t);
  if (warp == n_consumers) {
    // ---- producer: one thread keeps the ring full
    if (lane == 0) {
      const uint32_t* ev_src = p.events + L.ev_off + pair0;
      for (int rb = 0; rb < n_blocks; ++rb) {
        const int stage = rb % RR_STAGES;
        if (rb >= RR_STAGES && !mbar_wait(s_empty + stage, (uint32_t)(rb / RR_STAGES - 1) & 1u)) {
          atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          break;
        }
        mbar_arrive_expect_tx(s_full + stage, RR_TILE_BYTES + 2 * ev_bytes);
        const bool ff = rb < L.W_pre;
        tma_load_2d(s_tiles + (size_t)stage * RR_STAGE_BYTES, ff ? &p.map_ff[l] : &p.map_rec[l], col0,
                    (ff ? rb : rb - L.W_pre) * RR_ROWS, s_full + stage);
        uint32_t* const dst = s_ev + (size_t)stage * 2 * p.pb;
        bulk_load(dst, ev_src + (size_t)rb * p.ev_stride, ev_bytes, s_full + stage);
        bulk_load(dst + p.pb, ev_src + p.raw_off + (size_t)rb * p.ev_stride, ev_bytes, s_full + stage);
      }
    }
    return;   // copies still in flight complete on barriers the consumers wait for before they leave
  }
  // ---- consumers
  unsigned long long acc01[RR_PPW], acc23[RR_PPW];
#pragma unroll
  for (int i = 0; i < RR_PPW; ++i) acc01[i] = acc23[i] = 0ull;   // +0.0f in both halves
  const uint32_t lane_off = smem_u32(s_tiles) + (uint32_t)lane * 16u;
  for (int rb = 0; rb < n_blocks; ++rb) {
    const int stage = rb % RR_STAGES;
    if (!mbar_wait(s_full + stage, (uint32_t)(rb / RR_STAGES) & 1u)) {
      if (lane == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      return;
    }
    const uint32_t tile = lane_off + (uint32_t)stage * RR_STAGE_BYTES;
    const uint32_t* const evs = s_ev + (size_t)stage * 2 * p.pb + warp * RR_PPW;
    uint32_t e[RR_PPW];
#pragma unroll
    for (int i = 0; i < RR_PPW / 4; ++i) {
      const uint4 x = reinterpret_cast<const uint4*>(evs)[i];
      e[4 * i] = x.x; e[4 * i + 1] = x.y; e[4 * i + 2] = x.z; e[4 * i + 3] = x.w;
    }
    // one event: the row's 16 bytes of this lane, two packed additions
    auto add_row = [&](int i, uint32_t r) {
      unsigned long long w01, w23;
      lds_2x64(tile + r * (RR_COLS * 4u), w01, w23);
      add_f32x2(acc01[i], w01); add_f32x2(acc23[i], w23);
    };
    // One row per pair without a look at the count (a missing row is the row of zeros): eight independent reads in
    // flight, no branch.  The second row, the third and fourth, or the rows of a block with more than four (raw spike
    // word, its two lowest bits already done) follow behind branches on the count, which is the same for the whole
    // warp.  Per accumulator the rows are added in ascending order.  (Measured per recomputation pass of the largest
    // benchmark network: two unconditional rows 77 ms, one 68 ms, none 69 ms: the kernel is bound by shared-memory reads,
    // and at 5 % activity a block of 32 rows holds no event in 22 % of the pairs and one in 34 %.)
#pragma unroll
    for (int i = 0; i < RR_PPW; ++i) add_row(i, (e[i] >> 8) & 0xffu);
#pragma unroll
    for (int i = 0; i < RR_PPW; ++i) {
      const uint32_t cnt = e[i] & 7u;
      if (cnt > 1) add_row(i, (e[i] >> 16) & 0xffu);
      if (cnt > 2) {   // the second word of the pair is read only here: one block in five has more than two events
        const uint32_t rw = evs[p.pb + i];
        if (cnt != RR_EV_MANY) {
          add_row(i, rw & 0xffu);
          add_row(i, (rw >> 8) & 0xffu);
        } else {
          uint32_t bits = rw;
          bits &= bits - 1;
          bits &= bits - 1;
          while (bits) {
            add_row(i, (uint32_t)__ffs(bits) - 1u);
            bits &= bits - 1;
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(s_empty + stage);
  }
  const int col = col0 + lane * 4;
  if (col < L.N) {
#pragma unroll
    for (int i = 0; i < RR_PPW; ++i) {
      const int pair = pair0 + warp * RR_PPW + i;
      if (pair < pairs) {
        const int d = p.d0 + 1 + pair / p.B, b = pair % p.B;
        float4 v;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(acc01[i]));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(v.z), "=f"(v.w) : "l"(acc23[i]));
        *reinterpret_cast<float4*>(p.slots + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride + L.state_off +
                                   (size_t)b * L.N + col) = v;
      }
    }
  }
}

// The same for the graded cell: an event carries a value, and an accumulator takes fma(value, w, acc) per event in
// the same ascending order.  The pre-pass stores, per (block of 32 rows, pair), the count, up to eight row numbers
// (two words, one byte each) and the eight values that go with them (read from the value pool at the position the
// stored list offsets and per-word prefixes give); a block with more events keeps its raw spike word and the pool
// position of its first value, and the consumer reads those values from the pool.
struct RowsGradedLayer {
  const uint32_t* ff_off;     // list offsets of the layer below, row 0: [(T+2)][B]
  const uint16_t* ff_pref;    // events before each spike word of the layer below, row 0: [(T+2)][B][W_pre]
  const float* ff_vals;       // its value pool [B][ff_cap]
  const uint32_t* rec_off;    // the same for the own layer
  const uint16_t* rec_pref;
  const float* rec_vals;
  size_t ff_cap, rec_cap;
};

struct RowsGradedParams {
  RowsParams r;               // events: plane 0 counts, 1 and 2 row numbers, 3 .. 10 values [block][pair][8]
  RowsGradedLayer g[MAXL];
  size_t plane;               // words per plane
};

constexpr uint32_t RRG_MAX = 8;        // events of a block held in the staged words
constexpr uint32_t RRG_MANY = 15u;     // count of a block with more
__host__ __device__ inline size_t refwd_rows_graded_smem_bytes(int pb) {
  return (size_t)RR_STAGES * (RR_TILE_BYTES + 11 * (size_t)pb * sizeof(uint32_t)) + 2 * RR_STAGES * sizeof(uint64_t);
}

__global__ void __launch_bounds__(128) rows_events_graded_kernel(const __grid_constant__ RowsGradedParams gp) {
  pdl_launch_dependents();
  const RowsParams& p = gp.r;
  const RowsLayer& L = p.lay[blockIdx.z];
  const RowsGradedLayer& G = gp.g[blockIdx.z];
  const int rb = blockIdx.y, pair = blockIdx.x * 128 + threadIdx.x;
  if (rb >= L.W_pre + L.W || pair >= p.ev_stride) return;
  pdl_wait();
  uint32_t bits = 0;
  uint32_t first = 0;          // position of the block's first value in its sample's pool
  const float* pool = G.ff_vals;   // ... which starts here
  if (pair < p.n * p.B) {
    const int t = p.t0 + p.d0 + 1 + pair / p.B, b = pair % p.B;
    if (rb < L.W_pre) {
      const size_t row = (size_t)(t - L.ff_row0) * p.B + b;        // spike words of the layer below at step t
      bits = L.ff_words[row * L.W_pre + rb];
      if (rb == L.W_pre - 1) bits &= last_word_mask(L.N_pre);
      const size_t lrow = (size_t)t * p.B + b;                      // its list (step t) in the offset and prefix rows
      first = G.ff_off[lrow] + G.ff_pref[lrow * L.W_pre + rb];
      pool = G.ff_vals + (size_t)b * G.ff_cap;
    } else {
      const size_t lrow = (size_t)(t - 1) * p.B + b;                // own layer at step t - 1
      bits = L.words[lrow * L.W + (rb - L.W_pre)];
      first = G.rec_off[lrow] + G.rec_pref[lrow * L.W + (rb - L.W_pre)];
      pool = G.rec_vals + (size_t)b * G.rec_cap;
    }
  }
  const uint32_t cnt = __popc(bits);
  const size_t at = L.ev_off + (size_t)rb * p.ev_stride + pair;
  uint32_t ra = bits, rbw = first;   // more than RRG_MAX events: the raw word and the position in the sample's pool
  float v[RRG_MAX];
#pragma unroll
  for (int k = 0; k < (int)RRG_MAX; ++k) v[k] = 0.f;
  if (cnt <= RRG_MAX) {
    ra = 0; rbw = 0;
    uint32_t rest = bits;
#pragma unroll
    for (int k = 0; k < (int)RRG_MAX; ++k) {
      if (rest) {
        const uint32_t r = (uint32_t)(__ffs(rest) - 1);
        rest &= rest - 1;
        if (k < 4) ra |= r << (8 * k); else rbw |= r << (8 * (k - 4));
        v[k] = pool[first + k];
      }
    }
  }
  p.events[at] = cnt <= RRG_MAX ? cnt : RRG_MANY;
  p.events[gp.plane + at] = ra;
  p.events[2 * gp.plane + at] = rbw;
  float4* vdst = reinterpret_cast<float4*>(p.events + 3 * gp.plane + 8 * at);
  vdst[0] = make_float4(v[0], v[1], v[2], v[3]);
  vdst[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// a = fma(v, w, a) on two fp32 lanes, each rounded once (as __fmaf_rn)
__device__ __forceinline__ void fma_f32x2(unsigned long long& a, const unsigned long long w, const unsigned long long vv) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a) : "l"(w), "l"(vv));
}

__global__ void __launch_bounds__(32 * (RR_MAX_PB / RR_PPW + 1)) refwd_rows_graded_kernel(const __grid_constant__ RowsGradedParams gp) {
  pdl_launch_dependents();
  const RowsParams& p = gp.r;
  const int l = blockIdx.z;
  const RowsLayer& L = p.lay[l];
  const RowsGradedLayer& G = gp.g[l];
  const int col0 = blockIdx.y * RR_COLS;
  const int pairs = p.n * p.B, pair0 = blockIdx.x * p.pb;
  if (col0 >= L.N || pair0 >= pairs) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_consumers = p.pb / RR_PPW;
  extern __shared__ __align__(128) unsigned char s_raw_bytes[];
  float4* const s_tiles = reinterpret_cast<float4*>(s_raw_bytes);                                         // [RR_STAGES][32][32]
  uint32_t* const s_ev = reinterpret_cast<uint32_t*>(s_raw_bytes + (size_t)RR_STAGES * RR_TILE_BYTES);   // [RR_STAGES][11][pb]
  uint64_t* const s_full = reinterpret_cast<uint64_t*>(s_ev + (size_t)RR_STAGES * 11 * p.pb);
  uint64_t* const s_empty = s_full + RR_STAGES;
  const int n_blocks = L.W_pre + L.W;
  if (tid == 0) {
    for (int s = 0; s < RR_STAGES; ++s) { mbar_init(s_full + s, 1); mbar_init(s_empty + s, n_consumers); }
    mbar_fence_init();
  }
  __syncthreads();
  pdl_wait();
  const uint32_t ev_bytes = (uint32_t)p.pb * sizeof(uint32_t);
  if (warp == n_consumers) {
    if (lane == 0) {
      const uint32_t* ev_src = p.events + L.ev_off + pair0;
      for (int rb = 0; rb < n_blocks; ++rb) {
        const int stage = rb % RR_STAGES;
        if (rb >= RR_STAGES && !mbar_wait(s_empty + stage, (uint32_t)(rb / RR_STAGES - 1) & 1u)) {
          atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          break;
        }
        mbar_arrive_expect_tx(s_full + stage, RR_TILE_BYTES + 11 * ev_bytes);
        const bool ff = rb < L.W_pre;
        tma_load_2d(s_tiles + (size_t)stage * (RR_TILE_BYTES / 16), ff ? &p.map_ff[l] : &p.map_rec[l], col0,
                    (ff ? rb : rb - L.W_pre) * RR_ROWS, s_full + stage);
        uint32_t* const dst = s_ev + (size_t)stage * 11 * p.pb;
        const uint32_t* const src = ev_src + (size_t)rb * p.ev_stride;
        bulk_load(dst, src, ev_bytes, s_full + stage);
        bulk_load(dst + p.pb, src + gp.plane, ev_bytes, s_full + stage);
        bulk_load(dst + 2 * p.pb, src + 2 * gp.plane, ev_bytes, s_full + stage);
        bulk_load(dst + 3 * p.pb, p.events + 3 * gp.plane + 8 * (L.ev_off + (size_t)rb * p.ev_stride + pair0), 8 * ev_bytes,
                  s_full + stage);
      }
    }
    return;
  }
  unsigned long long acc01[RR_PPW], acc23[RR_PPW];
#pragma unroll
  for (int i = 0; i < RR_PPW; ++i) acc01[i] = acc23[i] = 0ull;
  const uint32_t lane_off = smem_u32(s_tiles) + (uint32_t)lane * 16u;
  for (int rb = 0; rb < n_blocks; ++rb) {
    const int stage = rb % RR_STAGES;
    if (!mbar_wait(s_full + stage, (uint32_t)(rb / RR_STAGES) & 1u)) {
      if (lane == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      return;
    }
    const uint32_t tile = lane_off + (uint32_t)stage * RR_TILE_BYTES;
    const uint32_t* const evs = s_ev + (size_t)stage * 11 * p.pb + warp * RR_PPW;
    const float* const vals = reinterpret_cast<const float*>(s_ev + (size_t)stage * 11 * p.pb + 3 * p.pb) + warp * RR_PPW * 8;
    auto fma_row = [&](int i, uint32_t r, float v) {
      unsigned long long w01, w23, vv;
      lds_2x64(tile + r * (RR_COLS * 4u), w01, w23);
      asm("mov.b64 %0, {%1, %1};" : "=l"(vv) : "f"(v));
      fma_f32x2(acc01[i], w01, vv); fma_f32x2(acc23[i], w23, vv);
    };
#pragma unroll
    for (int i = 0; i < RR_PPW; ++i) {
      const uint32_t cnt = evs[i];
      if (cnt == 0) continue;
      if (cnt != RRG_MANY) {
        uint32_t rows = evs[p.pb + i];
        for (uint32_t k = 0; k < cnt; ++k) {   // ascending rows; the count is the same for the whole warp
          if (k == 4) rows = evs[2 * p.pb + i];
          fma_row(i, rows & 0xffu, vals[i * 8 + k]);
          rows >>= 8;
        }
      } else {
        uint32_t bits = evs[p.pb + i];
        const int b = (pair0 + warp * RR_PPW + i) % p.B;
        const float* src = rb < L.W_pre ? G.ff_vals + (size_t)b * G.ff_cap : G.rec_vals + (size_t)b * G.rec_cap;
        size_t at = evs[2 * p.pb + i];   // position of the block's first value in the sample's pool
        while (bits) {
          fma_row(i, (uint32_t)__ffs(bits) - 1u, __ldg(src + at));
          bits &= bits - 1;
          ++at;
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(s_empty + stage);
  }
  const int col = col0 + lane * 4;
  if (col < L.N) {
#pragma unroll
    for (int i = 0; i < RR_PPW; ++i) {
      const int pair = pair0 + warp * RR_PPW + i;
      if (pair < pairs) {
        const int d = p.d0 + 1 + pair / p.B, b = pair % p.B;
        float4 v;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(v.x), "=f"(v.y) : "l"(acc01[i]));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(v.z), "=f"(v.w) : "l"(acc23[i]));
        *reinterpret_cast<float4*>(p.slots + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride + L.state_off +
                                   (size_t)b * L.N + col) = v;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Forward pass over a whole segment of steps in one cooperative launch (LIF cell).
//
// Unlike the recomputation above the spikes are not known yet, so a CTA (column tile, sample b,
// layer l) can start step t only when the spike words of (l, t-1, b) and (l-1, t, b) are complete.
// These are the only dependences: samples never wait for one another and a lower layer may run
// ahead of a higher one.  Each (layer, sample) has a counter of finished (tile, step) pairs; a
// producer publishes its words with a release add to the counter, a consumer polls the counter with
// acquire loads and then reads the words past L1.  Every buffer a step writes is indexed by the
// step or owned by the writing thread, so running ahead overwrites nothing that is still needed.
// All CTAs must be resident together (cooperative launch); a wait that does not end within
// SYNC_POLL_LIMIT polls raises STATUS_SYNC_TIMEOUT and the CTA returns.
constexpr uint32_t SYNC_POLL_LIMIT = 1u << 22;   // a few seconds
constexpr int SEG_WORDS = 1024;                  // spike words of both sources of a layer, staged per step

struct FwdSegLayer {
  const float* W_ff;          // [N_pre][N]
  const float* W_rec;         // [N][N]
  const uint32_t* ff_words;   // spike words of the layer below; row of step t at (t - ff_row0) * B * W_pre
  uint32_t* words;            // own spike words [T+1][B][W]
  uint32_t* ff_pool;          // event pool of the layer below [B][ff_cap] (written here if write_ff_list)
  uint32_t* ff_off;           // its offsets, row 0
  uint32_t* rec_pool;         // own event pool [B][rec_cap]
  uint32_t* rec_off;          // own offsets, row 0
  uint32_t* counts;           // [B][N] spike counts (last layer) or null
  float* V_dbg;               // [T+1][B][N] copy of every state, or null
  size_t state_off;           // offset of this layer inside a state slot, in floats
  uint32_t ff_cap, rec_cap;
  int N_pre, N, W_pre, W;
  int ff_row0;                // 1 for the input (its rows start at step 1), 0 for hidden layers
  int write_ff_list;          // the layer below is the input: this layer stores its lists
  int tiles;                  // column tiles (CTAs per sample) of this layer
};

struct FwdSegParams {
  FwdSegLayer lay[MAXL];
  float* slots;
  size_t slot_stride;         // floats
  uint32_t* status;
  uint32_t* progress;         // [L][B] finished (tile, step) pairs, zero at launch
  int B, t0, t1;
  int in_slot, buf_slot, buf_len, keep_every, keep_slot;
  int ring_groups;            // groups of eight rows in the copy ring (dynamic shared memory: 16 KB each)
  float alpha, theta;
};

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Publishes one more finished (tile, step) pair.  Called by one thread after a CTA barrier: the release makes
// everything the CTA wrote before that barrier visible to whoever reads the new count with an acquire load.
__device__ __forceinline__ void publish_progress(uint32_t* counter) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(counter), "r"(1u) : "memory");
}

__device__ __forceinline__ bool wait_progress(const uint32_t* counter, uint32_t target,
                                              uint32_t poll_limit = SYNC_POLL_LIMIT) {
  for (uint32_t i = 0; i < poll_limit; ++i) {
    if (ld_acquire_gpu(counter) >= target) return true;
    if (i > 32) __nanosleep(64);
  }
  return false;
}

// The waiting protocol on its own, for a self-test: one CTA waits for a count that nobody publishes; the
// wait must give up after poll_limit polls, raise the status bit and let the kernel end.
__global__ void wait_selftest_kernel(uint32_t* status, const uint32_t* counter, uint32_t poll_limit) {
  __shared__ int s_ok;
  if (threadIdx.x == 0) {
    const bool ok = wait_progress(counter, 1u, poll_limit);
    if (!ok) atomicOr(status, STATUS_SYNC_TIMEOUT);
    s_ok = ok ? 1 : 0;
  }
  __syncthreads();
  if (!s_ok) return;
  status[1] = 1u;   // not reached unless somebody published
}

// The gather is that of fwd_step_kernel: a fifth warp copies the listed rows as bulk copies through a ring of groups
// of eight rows, the four consumer warps add them in list order.  The ring is as deep as the launch allows
// (FwdSegParams::ring_groups; one CTA per SM when the grid fits that way: a deep ring is what lets one SM gather from L2
// at more than the 45 GB/s that four warps of 16-byte copies reach).
constexpr int SEG_RING_MAX = 10;   // groups of eight rows in the ring at most (160 KB)

__global__ void __launch_bounds__(FWDS_THREADS) fwd_segment_kernel(const __grid_constant__ FwdSegParams p) {
  const int l = blockIdx.z;
  const FwdSegLayer& L = p.lay[l];
  const int col0 = blockIdx.x * FWD_COLS;
  if (col0 >= L.N) return;
  const int b = blockIdx.y, B = p.B, tid = threadIdx.x;
  const bool tile0 = blockIdx.x == 0;
  __shared__ const float* s_row[LIST_CHUNK];
  __shared__ uint32_t s_words[SEG_WORDS];
  __shared__ uint32_t s_pref[SEG_WORDS + 1];
  __shared__ uint32_t s_warp[FWDS_THREADS / 32];
  __shared__ int s_ok;
  __shared__ uint64_t s_full[SEG_RING_MAX], s_empty[SEG_RING_MAX];
  extern __shared__ float4 s_stage[];   // [ring_groups][GATHER_ROWS][FWD_THREADS]
  const bool producer = tid >= FWD_THREADS;        // the fifth warp
  const int col = col0 + tid * 4;
  const bool active = !producer && col < L.N;
  const int G = p.ring_groups;
  if (tid == 0) {
    for (int i = 0; i < G; ++i) { mbar_init(s_full + i, 1); mbar_init(s_empty + i, FWD_THREADS / 32); }
    mbar_fence_init();
  }
  __syncthreads();
  // ring position of the next group (both roles count the groups of all steps alike); bytes of a row segment
  int gc = 0, slot = 0;
  uint32_t round = 0;          // gc / G
  bool dead = false;           // a wait of this warp ran out: no more waiting, copying or adding
  const uint32_t row_bytes = (uint32_t)(L.N - col0 < FWD_COLS ? L.N - col0 : FWD_COLS) * sizeof(float);
  const float* const Wff_tile = L.W_ff + col0;
  const float* const Wrec_tile = L.W_rec + col0;
  uint32_t* const ff_pool = L.ff_pool + (size_t)b * L.ff_cap;
  uint32_t* const rec_pool = L.rec_pool + (size_t)b * L.rec_cap;
  float* const state = p.slots + L.state_off + (size_t)b * L.N + col;
  uint32_t* const my_progress = p.progress + (size_t)l * B + b;
  const uint32_t* const below_progress = l > 0 ? p.progress + (size_t)(l - 1) * B + b : nullptr;
  const uint32_t below_tiles = l > 0 ? (uint32_t)p.lay[l - 1].tiles : 0u;

  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (active) v = *reinterpret_cast<const float4*>(state + (size_t)p.in_slot * p.slot_stride);
  // where the next lists go in the pools (this CTA is the only writer of its sample's pools)
  uint32_t rec_end = 0, ff_end = 0;
  if (tile0) {
    rec_end = L.rec_off[(size_t)p.t0 * B + b];
    if (L.write_ff_list) ff_end = L.ff_off[(size_t)(p.t0 + 1) * B + b];
  }

  for (int t = p.t0 + 1; t <= p.t1; ++t) {
    const uint32_t d = (uint32_t)(t - p.t0);
    if (tid == 0) {
      bool ok = wait_progress(my_progress, (uint32_t)L.tiles * (d - 1));
      if (ok && l > 0) ok = wait_progress(below_progress, below_tiles * d);
      if (!ok) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    if (!s_ok) return;
    {
      const uint32_t* ffw = L.ff_words + ((size_t)(t - L.ff_row0) * B + b) * L.W_pre;
      const uint32_t* recw = L.words + ((size_t)(t - 1) * B + b) * L.W;
      for (int w = tid; w < L.W_pre + L.W; w += FWDS_THREADS) {
        const uint32_t x = __ldcg(w < L.W_pre ? ffw + w : recw + (w - L.W_pre));
        s_words[w] = w == L.W_pre - 1 ? x & last_word_mask(L.N_pre) : x;
      }
    }
    __syncthreads();
    const WordPair wp{s_words, L.W_pre, s_words + L.W_pre, L.W};
    const uint32_t total = prefix_popcounts<FWDS_THREADS>(wp, s_pref, s_warp);
    const uint32_t n_ff = s_pref[L.W_pre];
    const uint32_t pw = active ? s_words[L.W_pre + (col >> 5)] >> (col & 31) : 0u;
    if (tile0) {   // append the two lists to the event pools
      const bool wr_ff = L.write_ff_list != 0;
      const uint32_t room_ff = wr_ff ? L.ff_cap - ff_end : 0u, room_rec = L.rec_cap - rec_end;
      write_lists_from_words<FWDS_THREADS, false>(wp, s_pref, n_ff, wr_ff ? ff_pool + ff_end : nullptr, room_ff,
                                                 rec_pool + rec_end, room_rec);
      const uint32_t n_rec = total - n_ff;
      rec_end += n_rec < room_rec ? n_rec : room_rec;
      if (wr_ff) ff_end += n_ff < room_ff ? n_ff : room_ff;
      if (tid == 0) {
        L.rec_off[(size_t)t * B + b] = rec_end;
        if (wr_ff) L.ff_off[(size_t)(t + 1) * B + b] = ff_end;
        if (n_rec > room_rec || (wr_ff && n_ff > room_ff)) atomicOr(p.status, STATUS_EVENT_OVERFLOW);
      }
    }

    // gather-accumulate in list order: feed-forward events, then recurrent events
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t c0 = 0; c0 < total; c0 += LIST_CHUNK) {
      const int n = (int)(total - c0 < (uint32_t)LIST_CHUNK ? total - c0 : (uint32_t)LIST_CHUNK);
      fill_rows_from_words<FWDS_THREADS>(wp, s_pref, c0, Wff_tile, Wrec_tile, L.N, s_row);
      __syncthreads();
      const int n_groups = (n + GATHER_ROWS - 1) / GATHER_ROWS;
      if (producer) {
        // ---- producer warp
        gather_producer(s_row, n, reinterpret_cast<unsigned char*>(s_stage), G, s_full, s_empty, row_bytes, gc, dead, p.status,
                        FWDS_GROUP_BYTES, FWDS_ROW_BYTES);
      } else {
        // ---- consumers: the rows of a group in list order
        for (int g = 0; g < n_groups && !dead; ++g) {
          if (!mbar_wait(s_full + slot, round & 1u)) {
            if ((tid & 31) == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
            dead = true;
            break;
          }
          if (active) {
            const float4* src = s_stage + (size_t)slot * GATHER_ROWS * FWD_THREADS + tid;
#pragma unroll
            for (int u = 0; u < GATHER_ROWS; ++u) {
              if (g * GATHER_ROWS + u < n) {
                const float4 w = src[u * FWD_THREADS];
                acc.x = __fadd_rn(acc.x, w.x); acc.y = __fadd_rn(acc.y, w.y);
                acc.z = __fadd_rn(acc.z, w.z); acc.w = __fadd_rn(acc.w, w.w);
              }
            }
          }
          __syncwarp();
          if ((tid & 31) == 0) mbar_arrive(s_empty + slot);
          ++gc;
          if (++slot == G) { slot = 0; ++round; }
        }
      }
      __syncthreads();
    }

    // leak, reset by subtraction of the previous step's own spike, threshold
    uint32_t nib = 0;
    if (active) {
      v.x = __fsub_rn(__fmaf_rn(p.alpha, v.x, acc.x), __fmul_rn(p.theta, (float)(pw & 1u)));
      v.y = __fsub_rn(__fmaf_rn(p.alpha, v.y, acc.y), __fmul_rn(p.theta, (float)((pw >> 1) & 1u)));
      v.z = __fsub_rn(__fmaf_rn(p.alpha, v.z, acc.z), __fmul_rn(p.theta, (float)((pw >> 2) & 1u)));
      v.w = __fsub_rn(__fmaf_rn(p.alpha, v.w, acc.w), __fmul_rn(p.theta, (float)((pw >> 3) & 1u)));
      *reinterpret_cast<float4*>(state + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride) = v;
      if (p.keep_every > 0 && d % p.keep_every == 0)
        *reinterpret_cast<float4*>(state + (size_t)(p.keep_slot + d / p.keep_every - 1) * p.slot_stride) = v;
      if (L.V_dbg) *reinterpret_cast<float4*>(L.V_dbg + ((size_t)t * B + b) * L.N + col) = v;
      nib = (v.x > p.theta ? 1u : 0u) | (v.y > p.theta ? 2u : 0u) | (v.z > p.theta ? 4u : 0u) |
            (v.w > p.theta ? 8u : 0u);
      if (L.counts && nib) {
        uint4* c = reinterpret_cast<uint4*>(L.counts + (size_t)b * L.N + col);
        uint4 cv = *c;
        cv.x += nib & 1u; cv.y += (nib >> 1) & 1u; cv.z += (nib >> 2) & 1u; cv.w += (nib >> 3) & 1u;
        *c = cv;
      }
    }
    if (!producer) {   // eight neighbouring lanes hold the 32 bits of one spike word
      const int lane = tid & 31;
      uint32_t word = nib << (4 * (lane & 7));
      word |= __shfl_xor_sync(0xffffffffu, word, 1);
      word |= __shfl_xor_sync(0xffffffffu, word, 2);
      word |= __shfl_xor_sync(0xffffffffu, word, 4);
      const int widx = col >> 5;
      if ((lane & 7) == 0 && widx < L.W) L.words[((size_t)t * B + b) * L.W + widx] = word;
    }
    __syncthreads();
    if (tid == 0) {   // publish: this tile's words of step t are complete
      publish_progress(my_progress);
    }
  }
  if (producer && dead)   // the copies of the last groups issued may still be on their way: wait for them, briefly
    for (int cc = gc > G ? gc - G : 0; cc < gc; ++cc) mbar_wait(s_full + cc % G, (uint32_t)(cc / G) & 1u, 1u << 14);
}

// ------------------------------------------------------------------------------------------
// Forward pass with the weights resident in shared memory (LIF cell, networks of a few thousand
// neurons: all weight matrices together must fit the shared memory of the whole device).
//
// A CTA owns RS_COLS columns of one layer and keeps those columns of W_ff and W_rec (every row) in
// shared memory for all steps of the launch, so an event costs a shared-memory read instead of an
// L2 gather.  Per step a half-warp turns the spike words of one sample into the list of weight rows
// in canonical order (feed-forward events, then recurrent ones, ascending); then the first eight
// warps add the rows, one thread per sample and two columns, apply leak, reset and threshold, and
// publish 16 spike bits per sample.  The event pools of a sample are appended to by one CTA of the
// layer (sample index modulo the number of CTAs).  Every CTA of a layer needs the words of all
// columns, so the layers synchronise through one counter each (finished (CTA, step) pairs), with
// the publish / poll protocol of fwd_segment_kernel.  Cooperative launch; bounded waits.
constexpr int RS_COLS = 16;        // columns of a layer per CTA
constexpr int RS_THREADS = 512;    // 32 half-warps: one per sample of a group
constexpr int RS_ADDERS = 256;     // threads that add rows: 32 samples x 8 column pairs
constexpr int RS_LIST = 256;       // list entries per sample staged at a time
constexpr int RS_MAX_GROUPS = 2;   // groups of 32 samples a thread can own: B <= 64

struct ResLayer {
  const float* W_ff;          // [N_pre][N]
  const float* W_rec;         // [N][N]
  const uint32_t* ff_words;   // spike words of the layer below; row of step t at (t - ff_row0) * B * W_pre
  uint32_t* words;            // own spike words [T+1][B][W]
  uint32_t* ff_pool;          // event pool of the layer below [B][ff_cap] (written here if write_ff_list)
  uint32_t* ff_off;           // its offsets, row 0
  uint32_t* rec_pool;         // own event pool [B][rec_cap]
  uint32_t* rec_off;          // own offsets, row 0
  uint32_t* counts;           // [B][N] spike counts (last layer) or null
  float* V_dbg;               // [T+1][B][N] copy of every state, or null
  size_t state_off;           // offset of this layer inside a state slot, in floats
  uint32_t ff_cap, rec_cap;
  int N_pre, N, W_pre, W;
  int ff_row0;                // 1 for the input (its rows start at step 1), 0 for hidden layers
  int write_ff_list;          // the layer below is the input: this layer stores its lists
  int tiles;                  // CTAs of this layer
  int cta0;                   // blockIdx.x of its first CTA
};

struct ResParams {
  ResLayer lay[MAXL];
  float* slots;
  size_t slot_stride;         // floats
  uint32_t* status;
  uint32_t* progress;         // [L] finished (CTA, step) pairs per layer, zero at launch
  int L, B, t0, t1;
  int in_slot, buf_slot, buf_len, keep_every, keep_slot;
  float alpha, theta;
};

__host__ __device__ inline size_t resident_words_bytes(int W_pre, int W, int B) {
  return ((size_t)B * (W_pre + W) * 4 + 15) / 16 * 16;
}
__host__ __device__ inline size_t resident_smem_bytes(int N_pre, int N, int W_pre, int W, int B) {
  return (size_t)(N_pre + N) * RS_COLS * 4 + resident_words_bytes(W_pre, W, B) + (size_t)32 * RS_LIST * 2;
}

__global__ void __launch_bounds__(RS_THREADS, 1) fwd_resident_kernel(const __grid_constant__ ResParams p) {
  int l = 0;
  while (l + 1 < p.L && (int)blockIdx.x >= p.lay[l + 1].cta0) ++l;
  const ResLayer& L = p.lay[l];
  const int tile = (int)blockIdx.x - L.cta0, col0 = tile * RS_COLS;
  const int tid = threadIdx.x, B = p.B;
  const int Wtot = L.W_pre + L.W, rows = L.N_pre + L.N;
  const int groups = (B + 31) / 32;
  extern __shared__ float4 s_dyn[];
  float* const Ws = reinterpret_cast<float*>(s_dyn);                                     // [rows][RS_COLS]
  uint32_t* const s_words = reinterpret_cast<uint32_t*>(Ws + (size_t)rows * RS_COLS);   // [B][Wtot]
  uint16_t* const s_list = reinterpret_cast<uint16_t*>(reinterpret_cast<char*>(s_words) +
                                                       resident_words_bytes(L.W_pre, L.W, B));   // [32][RS_LIST]
  __shared__ int s_ok;
  __shared__ int s_n[32];   // list entries of each of the 32 samples in this chunk
  __shared__ uint32_t s_ends[32][3];   // per sample: end of its recurrent and feed-forward pool lists, feed-forward events now

  // Two roles.  Compaction: half-warp `bl` (16 lanes, lane index c) turns the words of sample 32 gi + bl into
  // its list.  Accumulation: the first 256 threads; thread (sb, pair) owns columns 2 pair, 2 pair + 1 of
  // sample 32 gi + sb (eight warps: two per scheduler hide the shared-memory latency of one another).
  const int c = tid & (RS_COLS - 1), bl = tid >> 4;
  const bool adder = tid < RS_ADDERS;
  const int sb = tid >> 3, pair = tid & 7;
  const int acol = col0 + pair * 2;            // first of this thread's two columns (accumulation role)
  const bool acol_ok = adder && acol < L.N;    // N is even: both or none

  // ---- this CTA's columns of both matrices, every row, once per launch
  for (int q = tid; q < rows * (RS_COLS / 4); q += RS_THREADS) {
    const int r = q / (RS_COLS / 4), part = q % (RS_COLS / 4);
    const int cc = col0 + part * 4;
    const float* src = r < L.N_pre ? L.W_ff + (size_t)r * L.N + cc : L.W_rec + (size_t)(r - L.N_pre) * L.N + cc;
    cp_async16_or_zero(Ws + (size_t)r * RS_COLS + part * 4, cc < L.N ? src : L.W_ff, cc < L.N);
  }
  cp_async_commit();

  float2 v[RS_MAX_GROUPS];
  uint2 fired[RS_MAX_GROUPS];   // spikes of this thread's two neurons during this launch (last layer: for the readout)
  uint32_t rec_end[RS_MAX_GROUPS], ff_end[RS_MAX_GROUPS];
  bool owner[RS_MAX_GROUPS];   // this CTA appends the lists of the half-warp's sample to the event pools
#pragma unroll
  for (int gi = 0; gi < RS_MAX_GROUPS; ++gi) {
    v[gi] = make_float2(0.f, 0.f); fired[gi] = make_uint2(0u, 0u); rec_end[gi] = 0; ff_end[gi] = 0; owner[gi] = false;
    if (gi < groups) {
      const int ba = gi * 32 + sb, bc = gi * 32 + bl;
      if (acol_ok && ba < B)
        v[gi] = *reinterpret_cast<const float2*>(p.slots + (size_t)p.in_slot * p.slot_stride + L.state_off +
                                                 (size_t)ba * L.N + acol);
      owner[gi] = bc < B && bc % L.tiles == tile;
      if (owner[gi]) {
        rec_end[gi] = L.rec_off[(size_t)p.t0 * B + bc];
        if (L.write_ff_list) ff_end[gi] = L.ff_off[(size_t)(p.t0 + 1) * B + bc];
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();

  uint32_t* const my_progress = p.progress + l;
  const int wpl = (Wtot + RS_COLS - 1) / RS_COLS;   // words per lane of a half-warp
  uint16_t* const lst = s_list + (size_t)bl * RS_LIST;

  for (int t = p.t0 + 1; t <= p.t1; ++t) {
    const uint32_t d = (uint32_t)(t - p.t0);
    if (tid == 0) {
      bool ok = wait_progress(my_progress, (uint32_t)L.tiles * (d - 1));
      if (ok && l > 0) ok = wait_progress(p.progress + (l - 1), (uint32_t)p.lay[l - 1].tiles * d);
      if (!ok) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    if (!s_ok) return;

#pragma unroll
    for (int gi = 0; gi < RS_MAX_GROUPS; ++gi) {
      if (gi >= groups) break;                       // uniform
      // ---- compaction role
      const int b = gi * 32 + bl;
      const bool b_ok = b < B;
      uint32_t* const wrow = s_words + (size_t)(b_ok ? b : B - 1) * Wtot;
      if (b_ok) {   // the sample's spike words, past L1 (other CTAs wrote them during this launch)
        const uint32_t* ffw = L.ff_words + ((size_t)(t - L.ff_row0) * B + b) * L.W_pre;
        const uint32_t* recw = L.words + ((size_t)(t - 1) * B + b) * L.W;
        for (int w0 = c; w0 < Wtot; w0 += 4 * RS_COLS) {   // four loads in flight per lane
          uint32_t r[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int w = w0 + j * RS_COLS;
            r[j] = w < Wtot ? __ldcg(w < L.W_pre ? ffw + w : recw + (w - L.W_pre)) : 0u;
            if (w == L.W_pre - 1) r[j] &= last_word_mask(L.N_pre);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (w0 + j * RS_COLS < Wtot) wrow[w0 + j * RS_COLS] = r[j];
        }
      }
      __syncwarp();
      // events before this lane's words, in the sample's canonical order
      const int w_lo = c * wpl, w_hi = min(Wtot, w_lo + wpl);
      uint32_t cnt = 0, cnt_ff = 0;
      for (int w = w_lo; w < w_hi; ++w) {
        const uint32_t k = b_ok ? __popc(wrow[w]) : 0u;
        cnt += k;
        if (w < L.W_pre) cnt_ff += k;
      }
      uint32_t incl = cnt;
#pragma unroll
      for (int s = 1; s < RS_COLS; s <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, s, RS_COLS);
        if (c >= s) incl += y;
      }
      const uint32_t n_tot = __shfl_sync(0xffffffffu, incl, RS_COLS - 1, RS_COLS);
      uint32_t n_ff = cnt_ff;
#pragma unroll
      for (int s = RS_COLS / 2; s >= 1; s >>= 1) n_ff += __shfl_xor_sync(0xffffffffu, n_ff, s, RS_COLS);
      const uint32_t first = incl - cnt;
      const bool pools = owner[gi];
      const uint32_t room_rec = L.rec_cap - rec_end[gi], room_ff = L.write_ff_list ? L.ff_cap - ff_end[gi] : 0u;

      float2 acc = make_float2(0.f, 0.f);
      for (uint32_t c0 = 0;; c0 += RS_LIST) {
        // this lane's events that fall into [c0, c0 + RS_LIST): row of Ws into the list, index into the pools
        uint32_t pos = first;
        if (n_tot <= (uint32_t)RS_LIST) {   // the usual case: the whole list fits, no window to test against
          for (int w = w_lo; w < w_hi; ++w) {
            uint32_t bits = b_ok ? wrow[w] : 0u;
            const uint32_t idx0 = w < L.W_pre ? (uint32_t)w * 32u : (uint32_t)(w - L.W_pre) * 32u + (uint32_t)L.N_pre;
            while (bits) {
              lst[pos++] = (uint16_t)(idx0 + (uint32_t)(__ffs(bits) - 1));
              bits &= bits - 1;
            }
          }
        } else {
          for (int w = w_lo; w < w_hi && pos < c0 + RS_LIST; ++w) {
            uint32_t bits = b_ok ? wrow[w] : 0u;
            const uint32_t idx0 = w < L.W_pre ? (uint32_t)w * 32u : (uint32_t)(w - L.W_pre) * 32u + (uint32_t)L.N_pre;
            if (pos + __popc(bits) <= c0) { pos += __popc(bits); continue; }
            while (bits) {
              const uint32_t idx = idx0 + (uint32_t)(__ffs(bits) - 1);
              bits &= bits - 1;
              if (pos >= c0 && pos < c0 + RS_LIST) lst[pos - c0] = (uint16_t)idx;
              ++pos;
            }
          }
        }
        if (c == 0) {
          s_n[bl] = (int)(n_tot > c0 ? (n_tot - c0 < (uint32_t)RS_LIST ? n_tot - c0 : (uint32_t)RS_LIST) : 0u);
          if (pools) { s_ends[bl][0] = rec_end[gi]; s_ends[bl][1] = ff_end[gi]; s_ends[bl][2] = n_ff; }
        }
        const int more = __syncthreads_or(n_tot > c0 + RS_LIST);   // the lists of all 32 samples are in place
        // ---- accumulation role: in list order, one accumulator per (sample, column)
        if (adder) {
          const int n = s_n[sb];
          const uint16_t* const al = s_list + (size_t)sb * RS_LIST;
          const float2* const Wp = reinterpret_cast<const float2*>(Ws) + pair;
          auto add2 = [&](const float2 r) { acc.x = __fadd_rn(acc.x, r.x); acc.y = __fadd_rn(acc.y, r.y); };
          // eight rows at a time, the next eight already on their way while these are added
          auto load8 = [&](int e, float2 (&w)[8]) {
            const uint4 pk = *reinterpret_cast<const uint4*>(al + e);
            w[0] = Wp[(pk.x & 0xffffu) * (RS_COLS / 2)]; w[1] = Wp[(pk.x >> 16) * (RS_COLS / 2)];
            w[2] = Wp[(pk.y & 0xffffu) * (RS_COLS / 2)]; w[3] = Wp[(pk.y >> 16) * (RS_COLS / 2)];
            w[4] = Wp[(pk.z & 0xffffu) * (RS_COLS / 2)]; w[5] = Wp[(pk.z >> 16) * (RS_COLS / 2)];
            w[6] = Wp[(pk.w & 0xffffu) * (RS_COLS / 2)]; w[7] = Wp[(pk.w >> 16) * (RS_COLS / 2)];
          };
          auto add8 = [&](const float2 (&w)[8]) {
#pragma unroll
            for (int j = 0; j < 8; ++j) add2(w[j]);
          };
          const int n8 = n & ~7;
          float2 wa[8], wb[8];
          int e = 0;
          if (n8 > 0) load8(0, wa);
          while (e < n8) {
            if (e + 8 < n8) load8(e + 8, wb);
            add8(wa);
            e += 8;
            if (e >= n8) break;
            if (e + 8 < n8) load8(e + 8, wa);
            add8(wb);
            e += 8;
          }
          for (; e < n; ++e) {
            add2(Wp[(uint32_t)al[e] * (RS_COLS / 2)]);
          }
        } else {
          // ---- meanwhile the other warps append the lists of the samples this CTA owns to the event pools
          const int h = (tid - RS_ADDERS) >> 4, n_helpers = (RS_THREADS - RS_ADDERS) >> 4;
          int bb = tile;
          while (bb < 32 * gi) bb += L.tiles;
          for (int k = 0; bb < B && bb < 32 * gi + 32; bb += L.tiles, ++k) {
            if (k % n_helpers != h) continue;
            const int sl = bb & 31;
            const uint16_t* const pl = s_list + (size_t)sl * RS_LIST;
            const uint32_t r_end = s_ends[sl][0], f_end = s_ends[sl][1], nf = s_ends[sl][2];
            const uint32_t rm_rec = L.rec_cap - r_end, rm_ff = L.write_ff_list ? L.ff_cap - f_end : 0u;
            const int n = s_n[sl];
            for (int e = c; e < n; e += RS_COLS) {
              const uint32_t r = pl[e], pos = c0 + (uint32_t)e;
              if (pos < nf) { if (pos < rm_ff) L.ff_pool[(size_t)bb * L.ff_cap + f_end + pos] = r; }
              else if (pos - nf < rm_rec) L.rec_pool[(size_t)bb * L.rec_cap + r_end + (pos - nf)] = r - (uint32_t)L.N_pre;
            }
          }
        }
        if (!more) break;
        __syncthreads();   // before the lists are refilled
      }

      // ---- leak, reset by subtraction of the previous step's own spike, threshold (accumulation role)
      const int ba = gi * 32 + sb;
      uint32_t two = 0;
      if (acol_ok && ba < B) {
        const uint32_t pw = s_words[(size_t)ba * Wtot + L.W_pre + (acol >> 5)] >> (acol & 31);
        float2 vn;
        vn.x = __fsub_rn(__fmaf_rn(p.alpha, v[gi].x, acc.x), __fmul_rn(p.theta, (float)(pw & 1u)));
        vn.y = __fsub_rn(__fmaf_rn(p.alpha, v[gi].y, acc.y), __fmul_rn(p.theta, (float)((pw >> 1) & 1u)));
        v[gi] = vn;
        float* const st = p.slots + L.state_off + (size_t)ba * L.N + acol;
        *reinterpret_cast<float2*>(st + (size_t)(p.buf_slot + (d - 1) % p.buf_len) * p.slot_stride) = vn;
        if (p.keep_every > 0 && d % p.keep_every == 0)
          *reinterpret_cast<float2*>(st + (size_t)(p.keep_slot + d / p.keep_every - 1) * p.slot_stride) = vn;
        if (L.V_dbg) *reinterpret_cast<float2*>(L.V_dbg + ((size_t)t * B + ba) * L.N + acol) = vn;
        two = (vn.x > p.theta ? 1u : 0u) | (vn.y > p.theta ? 2u : 0u);
        fired[gi].x += two & 1u; fired[gi].y += (two >> 1) & 1u;
      }
      if (adder) {   // whole warps: eight neighbouring lanes hold the 16 spike bits of one sample
        uint32_t half = two << (2 * pair);
        half |= __shfl_xor_sync(0xffffffffu, half, 1);
        half |= __shfl_xor_sync(0xffffffffu, half, 2);
        half |= __shfl_xor_sync(0xffffffffu, half, 4);
        if (pair == 0 && ba < B) {
          uint16_t* const hrow = reinterpret_cast<uint16_t*>(L.words + ((size_t)t * B + ba) * L.W);
          hrow[tile] = (uint16_t)half;
          if (tile == L.tiles - 1 && (L.tiles & 1)) hrow[tile + 1] = 0;   // the unused half of the last word
        }
      }
      // ---- compaction role again: where this sample's lists now end
      if (pools && c == 0) {
        const uint32_t n_rec = n_tot - n_ff;
        rec_end[gi] += n_rec < room_rec ? n_rec : room_rec;
        L.rec_off[(size_t)t * B + b] = rec_end[gi];
        bool over = n_rec > room_rec;
        if (L.write_ff_list) {
          ff_end[gi] += n_ff < room_ff ? n_ff : room_ff;
          L.ff_off[(size_t)(t + 1) * B + b] = ff_end[gi];
          over = over || n_ff > room_ff;
        }
        if (over) atomicOr(p.status, STATUS_EVENT_OVERFLOW);
      }
      rec_end[gi] = __shfl_sync(0xffffffffu, rec_end[gi], 0, RS_COLS);   // the other lanes keep the same running ends
      ff_end[gi] = __shfl_sync(0xffffffffu, ff_end[gi], 0, RS_COLS);
      if (gi + 1 < groups) __syncthreads();   // s_list and s_n are reused by the next group of samples
    }
    __syncthreads();
    if (tid == 0) {   // publish: this CTA's spike bits of step t are complete
      publish_progress(my_progress);
    }
  }
  // spike counts of the launch into the time-summed counts the readout uses (this thread is their only writer)
  if (L.counts && acol_ok) {
#pragma unroll
    for (int gi = 0; gi < RS_MAX_GROUPS; ++gi) {
      const int ba = gi * 32 + sb;
      if (gi < groups && ba < B) {
        uint2* cp = reinterpret_cast<uint2*>(L.counts + (size_t)ba * L.N + acol);
        uint2 cv = *cp;
        cv.x += fired[gi].x; cv.y += fired[gi].y;
        *cp = cv;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Backward step: delta^l_t = g_S sigma'(V^l_t - theta) + alpha delta^l_{t+1}, with
// g_S = g_out + W_ff^{l+1} delta^{l+1}_t + W_rec^l delta^l_{t+1} - theta delta^l_{t+1}.
//
// A CTA owns 32 rows i of the two weight matrices: 8 row groups of 4 rows, one warp per
// (row group, group of BT samples).  The 32 lanes of a warp split the contraction index; a
// thread-block cluster of CS CTAs splits it further (rank r takes the r-th slice of each
// matrix).  Partial sums: per lane 4 x BT accumulators, reduced across the warp in a fixed
// tree that leaves each lane with its own (row, sample) totals, then across the cluster through
// distributed shared memory in rank order.  The order is fixed by (N, CS) alone.
struct BwdLayer {
  const float* W_rec;     // [N][N]
  const float* W_ffa;     // W_ff of the layer above [N][N_post] or null
  float* V_delta;         // [B][N]: V_t on entry, delta_t on exit
  const float* d_next;    // [B][N]      delta^l_{t+1}
  const float* d_above;   // [B][N_post] delta^{l+1}_t or null
  const float* g_out;     // [B][N] or null
  const float* g_ff;      // [B][N] or null: W_ff^{l+1} delta^{l+1}_t computed ahead for a run of steps, as
                          // g_ff_parts partial sums over slices of the contraction range, g_ff_stride floats apart
  size_t g_ff_stride;
  int g_ff_parts;
  float* carry_out;       // optional second copy of delta_t
  int N, N_post;
  int mode;               // 0 idle, 1 step
};

struct BwdParams {
  BwdLayer lay[MAXL];
  int B;
  float alpha, theta, beta;
  int surrogate, cell;
};

constexpr int BWD_RT = 4;                 // rows per thread
constexpr int BWD_WR = 8;                 // row groups (warps along rows) per CTA
constexpr int BWD_TM = BWD_RT * BWD_WR;   // rows per CTA

__device__ __forceinline__ float surrogate_grad(float v, float theta, float beta, int surrogate, int cell) {
  const float x = v - theta;
  if (cell == 1) return x > 0.f ? 1.f : 0.f;
  if (surrogate == 0) {
    const float d = fmaf(beta, fabsf(x), 1.f);
    return 1.f / (d * d);
  }
  if (surrogate == 2) {   // triangle with support |x| < 1 / beta
    const float u = fmaf(-beta, fabsf(x), 1.f);
    return u > 0.f ? beta * u : 0.f;
  }
  const float s = 1.f / (1.f + expf(-beta * x));
  return beta * s * (1.f - s);
}

// Sum over the warp of NV per-lane values; on return lane i holds the totals of values
// i * NV/32 .. (i+1) * NV/32 - 1 in v[0 .. NV/32).
template <int NV>
__device__ __forceinline__ void warp_transpose_reduce(float (&v)[NV], int lane) {
  int n = NV;
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const bool upper = (lane & s) != 0;
    const int half = n / 2;
#pragma unroll
    for (int j = 0; j < NV / 2; ++j) {
      if (j < half) {
        const float send = upper ? v[j] : v[j + half];
        const float keep = upper ? v[j + half] : v[j];
        v[j] = keep + __shfl_xor_sync(0xffffffffu, send, s);
      }
    }
    n = half;
  }
}

constexpr int BWD_STAGES = 4;   // chunks of the W and delta tiles in flight per CTA

// What the epilogue of one output element needs from global memory; fetched before the contraction starts
// so that the loads are long done when the sums arrive.
struct BwdPre { float dn, go, gf, v; };

__device__ __forceinline__ BwdPre bwd_prefetch(const BwdParams& p, const BwdLayer& L, int i, int b) {
  BwdPre r{0.f, 0.f, 0.f, 0.f};
  if (i >= L.N || b >= p.B) return r;
  const size_t k = (size_t)b * L.N + i;
  r.dn = L.d_next[k];
  r.go = L.g_out ? L.g_out[k] : 0.f;
  if (L.g_ff) {   // the partial sums in slice order
    r.gf = L.g_ff[k];
    for (int s = 1; s < L.g_ff_parts; ++s) r.gf += L.g_ff[(size_t)s * L.g_ff_stride + k];
  }
  r.v = L.V_delta[k];
  return r;
}

__device__ __forceinline__ void bwd_epilogue(const BwdParams& p, const BwdLayer& L, int i, int b, float sum,
                                             const BwdPre& pre) {
  if (i >= L.N || b >= p.B) return;
  const size_t k = (size_t)b * L.N + i;
  float g = sum + pre.go;
  if (L.g_ff) g += pre.gf;
  if (p.cell == 0) g = fmaf(-p.theta, pre.dn, g);
  const float sp = surrogate_grad(pre.v, p.theta, p.beta, p.surrogate, p.cell);
  const float dl = fmaf(g, sp, p.alpha * pre.dn);
  L.V_delta[k] = dl;
  if (L.carry_out) L.carry_out[k] = dl;
}

// The contraction itself runs on the tensor cores as a 3-pass TF32 product: every fp32 operand is
// split into hi = tf32(x) and lo = tf32(x - hi), and D += A_lo B_hi + A_hi B_lo + A_hi B_hi with fp32
// accumulation, which keeps the result at fp32 accuracy (the dropped lo*lo term is ~2^-22 relative).
constexpr int BWD_LD = 132;   // padded row length (floats) of the staged tiles: fragment loads hit 32 banks

// fp32 -> two tf32 pieces (10 mantissa bits each): hi = x with its 13 low mantissa bits cleared, lo = x - hi (exact
// in fp32: the cleared bits).  mma.sync reads only the 19 high bits of a tf32 operand (checked on the device: clearing
// the low bits of lo as well changes no result bit), so lo is passed as it is and the tensor core cuts it to tf32.
// Two operations at full rate per value; conversion instructions run at an eighth of it and would cost as much as the
// tensor-core work they feed.  hi + tf32(lo) differs from x by less than 2^-20 |x|.
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi));
}
// D(16x8) += A(16x8, row) * B(8x8, col); lane = 4 g + t holds A[g][t], A[g+8][t], A[g][t+4], A[g+8][t+4],
// B[t][g], B[t+4][g] and D[g][2t], D[g][2t+1], D[g+8][2t], D[g+8][2t+1].
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Row length (floats) of the staged W and delta tiles of the step kernels.  A lane reads 2 KS adjacent values
// of a row with one 64- or 128-bit load (KS = 16 / NWARP k-steps per warp and chunk); rows 8 (KS = 1) or 16
// (KS = 2) banks apart make those loads conflict-free.
__host__ __device__ constexpr int bwd_ld(int nwarp) { return nwarp == 8 ? 144 : 136; }

// One warp's share of a chunk of 128 contraction values: KS consecutive k-steps of 8, i.e. the 8 KS values from
// warp * 8 KS on.  Lane (g, t) loads, from each of its rows, the 2 KS adjacent values at 2 KS t with one vector
// load and splits each once; within k-step j the hardware's k slots t and t + 4 take values 2 j and 2 j + 1 of
// that group, for W and delta alike (the contraction does not care which k sits in which slot as long as both
// operands agree).  Wl / Dl: this lane's first value in row g of the W tile / the delta tile; further rows of W
// at multiples of 8 ldw (2 MT of them: MT tiles of 16 rows), further sample tiles at multiples of 8 ldd.  Per k-step three passes, small terms
// first; `between(phase)` runs after each pass (phases 0, 1, 2 of the first k-step are where callers issue the
// copies that refill a stage).
template <int NTN, int KS, int MT = 2, class Between>
__device__ __forceinline__ void warp_chunk_mma(float (&acc)[MT][NTN][4], const float* Wl, int ldw, const float* Dl,
                                               int ldd, Between&& between) {
  static_assert(KS == 1 || KS == 2, "one or two k-steps per warp and chunk");
  uint32_t wh[2 * MT][2 * KS], wlo[2 * MT][2 * KS], dh[NTN][2 * KS], dlo[NTN][2 * KS];
#pragma unroll
  for (int r = 0; r < 2 * MT; ++r) {
    float v[2 * KS];
    if (KS == 2) {
      const float4 x = *reinterpret_cast<const float4*>(Wl + (size_t)r * 8 * ldw);
      v[0] = x.x; v[1] = x.y; v[2 * KS - 2] = x.z; v[2 * KS - 1] = x.w;
    } else {
      const float2 x = *reinterpret_cast<const float2*>(Wl + (size_t)r * 8 * ldw);
      v[0] = x.x; v[1] = x.y;
    }
#pragma unroll
    for (int i = 0; i < 2 * KS; ++i) split_tf32(v[i], wh[r][i], wlo[r][i]);
  }
#pragma unroll
  for (int nt = 0; nt < NTN; ++nt) {
    float v[2 * KS];
    if (KS == 2) {
      const float4 x = *reinterpret_cast<const float4*>(Dl + (size_t)nt * 8 * ldd);
      v[0] = x.x; v[1] = x.y; v[2 * KS - 2] = x.z; v[2 * KS - 1] = x.w;
    } else {
      const float2 x = *reinterpret_cast<const float2*>(Dl + (size_t)nt * 8 * ldd);
      v[0] = x.x; v[1] = x.y;
    }
#pragma unroll
    for (int i = 0; i < 2 * KS; ++i) split_tf32(v[i], dh[nt][i], dlo[nt][i]);
  }
#pragma unroll
  for (int j = 0; j < KS; ++j) {
    uint32_t a_hi[MT][4], a_lo[MT][4], b_hi[NTN][2], b_lo[NTN][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {   // rows mt 16 + g (loaded row 2 mt) and mt 16 + g + 8 (loaded row 2 mt + 1)
      a_hi[mt][0] = wh[2 * mt][2 * j];     a_hi[mt][1] = wh[2 * mt + 1][2 * j];
      a_hi[mt][2] = wh[2 * mt][2 * j + 1]; a_hi[mt][3] = wh[2 * mt + 1][2 * j + 1];
      a_lo[mt][0] = wlo[2 * mt][2 * j];     a_lo[mt][1] = wlo[2 * mt + 1][2 * j];
      a_lo[mt][2] = wlo[2 * mt][2 * j + 1]; a_lo[mt][3] = wlo[2 * mt + 1][2 * j + 1];
    }
#pragma unroll
    for (int nt = 0; nt < NTN; ++nt) {
      b_hi[nt][0] = dh[nt][2 * j]; b_hi[nt][1] = dh[nt][2 * j + 1];
      b_lo[nt][0] = dlo[nt][2 * j]; b_lo[nt][1] = dlo[nt][2 * j + 1];
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt) mma_tf32(acc[mt][nt], a_lo[mt], b_hi[nt]);
    between(3 * j);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt) mma_tf32(acc[mt][nt], a_hi[mt], b_lo[nt]);
    between(3 * j + 1);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt) mma_tf32(acc[mt][nt], a_hi[mt], b_hi[nt]);
    between(3 * j + 2);
  }
}

// NTN = sample tiles of 8 per pass (BP = 8 NTN samples), NWARP warps per CTA; launched with cluster
// size CS along x: blockIdx.x = row_tile * CS + rank.  A CTA owns 32 rows x BP samples.  Chunks of
// 128 k of W [32][128] and delta [BP][128] stream through a BWD_STAGES-deep cp.async pipeline; within
// a chunk warp w multiplies the k-steps w, w + NWARP, ... (8 k each) for the whole tile, so every warp
// ends with a partial 32 x BP tile: the partials are summed in warp order through shared memory, then
// across the cluster in rank order.
template <int NTN, int NWARP>
__global__ void __launch_bounds__(32 * NWARP, NWARP == 8 ? 2 : 1) bwd_step_kernel(const __grid_constant__ BwdParams p) {
  constexpr int LD = bwd_ld(NWARP), KS = 16 / NWARP;
  constexpr int NT = 32 * NWARP, BP = 8 * NTN, ROWS = BWD_TM + BP, STAGE_F = ROWS * LD, TILE = BWD_TM * BP;
  constexpr int TS = BP + 8, TILEP = BWD_TM * TS;   // padded rows of the warps' partial tiles: 64-bit stores without bank conflicts
  constexpr int EPI = TILE / NT;                    // output elements a thread finishes at most (cluster of one)
  static_assert(TILE % NT == 0 && NWARP * TILEP <= BWD_STAGES * STAGE_F, "partial tiles fit the stages");
  pdl_launch_dependents();
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const BwdLayer& L = p.lay[blockIdx.z];
  if (L.mode == 0) return;                          // same for the whole cluster
  const int tile_row0 = (blockIdx.x / CS) * BWD_TM;
  if (tile_row0 >= L.N) return;                     // same for the whole cluster
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  __shared__ float s_part[TILE];
  extern __shared__ float4 s_dyn[];
  float* const s_tiles = reinterpret_cast<float*>(s_dyn);   // [BWD_STAGES][ROWS][LD]; later [NWARP][32][BP]
  // this rank's slice of each contraction range, in units of 4 floats
  const int q_rec = L.N / 4, q_ff = L.W_ffa ? L.N_post / 4 : 0;
  const int lo_rec = (int)((long long)q_rec * rank / CS) * 4, hi_rec = (int)((long long)q_rec * (rank + 1) / CS) * 4;
  const int lo_ff = (int)((long long)q_ff * rank / CS) * 4, hi_ff = (int)((long long)q_ff * (rank + 1) / CS) * 4;
  // chunks run over this rank's slice of W_ff(l+1) first, then of W_rec, k ascending
  const int it_ff = (hi_ff - lo_ff + 127) / 128, it_all = it_ff + (hi_rec - lo_rec + 127) / 128;
  const int rlast = L.N - 1, blast = p.B - 1;
  // Every thread copies the same ITER (row, 16-byte column) positions of each chunk; their global
  // addresses at k = 0 are worked out once per pass over the samples, so that issuing a chunk costs an
  // add, a compare and the copy per position.
  constexpr int ITER = ROWS * 32 / NT;
  static_assert(ROWS * 32 % NT == 0, "the staged tile divides evenly among the threads");
  pdl_wait();
  for (int bp0 = 0; bp0 < p.B; bp0 += BP) {
    BwdPre pre[EPI];
#pragma unroll
    for (int j = 0; j < EPI; ++j) {
      const int q = tid + j * NT, e = CS == 1 ? q : rank + CS * q;
      pre[j] = (e < TILE) ? bwd_prefetch(p, L, tile_row0 + e / BP, bp0 + e % BP) : BwdPre{0.f, 0.f, 0.f, 0.f};
    }
    const float* src_rec[ITER];
    const float* src_ff[ITER];
    int dst_off[ITER], kcol[ITER];
#pragma unroll
    for (int j = 0; j < ITER; ++j) {
      const int q = tid + j * NT, rr = q >> 5, c4 = q & 31;
      kcol[j] = 4 * c4;
      dst_off[j] = rr * LD + 4 * c4;
      if (rr < BWD_TM) {   // rows and samples past the end are clamped to the last valid one; never used
        const size_t row = tile_row0 + rr < rlast ? tile_row0 + rr : rlast;
        src_rec[j] = L.W_rec + row * L.N + 4 * c4;
        src_ff[j] = L.W_ffa ? L.W_ffa + row * L.N_post + 4 * c4 : nullptr;
      } else {
        const size_t b = bp0 + rr - BWD_TM < blast ? bp0 + rr - BWD_TM : blast;
        src_rec[j] = L.d_next + b * L.N + 4 * c4;
        src_ff[j] = L.d_above ? L.d_above + b * L.N_post + 4 * c4 : nullptr;
      }
    }
    // positions [j0, j1) of chunk `it`; the caller commits the group once all ITER positions are issued
    auto issue_part = [&](int it, int j0, int j1) {
      if (it < it_all) {
        const bool ff = it < it_ff;
        const int k0 = ff ? lo_ff + it * 128 : lo_rec + (it - it_ff) * 128;
        const int hi = ff ? hi_ff : hi_rec;
        float* st = s_tiles + (size_t)(it % BWD_STAGES) * STAGE_F;
#pragma unroll
        for (int j = 0; j < ITER; ++j) {
          if (j < j0 || j >= j1) continue;
          if (k0 + kcol[j] < hi) cp_async16(st + dst_off[j], (ff ? src_ff[j] : src_rec[j]) + k0);
          else *reinterpret_cast<float4*>(st + dst_off[j]) = make_float4(0.f, 0.f, 0.f, 0.f);   // past the slice
        }
      }
    };
    auto issue = [&](int it) {
      issue_part(it, 0, ITER);
      cp_async_commit();
    };
    float acc[2][NTN][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
    for (int it = 0; it < BWD_STAGES - 1; ++it) issue(it);
    for (int it = 0; it < it_all; ++it) {
      cp_async_wait<BWD_STAGES - 2>();   // this thread's copies of chunk `it` have landed
      __syncthreads();                   // ... everybody's have, and chunk it-1 has been consumed
      // The copies that refill the stage chunk it-1 used are issued between the tensor-core passes of this
      // warp's first k-step: copy instructions and mma instructions queue on different pipes, and in program
      // order one after the other they would take turns instead of overlapping.
      const int it_refill = it + BWD_STAGES - 1;
      const float* Ws = s_tiles + (size_t)(it % BWD_STAGES) * STAGE_F;
      const float* Ds = Ws + BWD_TM * LD;
      const int kl = warp * 8 * KS + 2 * KS * t;   // this lane's values of the chunk
      warp_chunk_mma<NTN, KS>(acc, Ws + g * LD + kl, LD, Ds + g * LD + kl, LD, [&](int phase) {
        if (phase == 0) issue_part(it_refill, 0, ITER / 3);
        else if (phase == 1) issue_part(it_refill, ITER / 3, 2 * ITER / 3);
        else if (phase == 2) { issue_part(it_refill, 2 * ITER / 3, ITER); cp_async_commit(); }
      });
    }
    cp_async_wait<0>();
    __syncthreads();   // the stages are free: they now hold the warps' partial tiles [NWARP][32][TS]
    {
      float* mine = s_tiles + (size_t)warp * TILEP;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt) {
          const int r = mt * 16 + g, c = nt * 8 + 2 * t;
          *reinterpret_cast<float2*>(mine + r * TS + c) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
          *reinterpret_cast<float2*>(mine + (r + 8) * TS + c) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
    }
    __syncthreads();
    if (CS == 1) {
#pragma unroll
      for (int j = 0; j < EPI; ++j) {
        const int e = tid + j * NT;
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) sum += s_tiles[(size_t)w * TILEP + (e / BP) * TS + e % BP];
        bwd_epilogue(p, L, tile_row0 + e / BP, bp0 + e % BP, sum, pre[j]);
      }
      __syncthreads();   // before the next pass refills the stages
    } else {
      // this rank's partial sums go straight into the shared memory of the rank that finishes the element
      // (element e belongs to rank e % CS), one slice per sending rank
      const int per = TILE / CS;
      for (int e = tid; e < TILE; e += NT) {
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) sum += s_tiles[(size_t)w * TILEP + (e / BP) * TS + e % BP];
        cluster.map_shared_rank(s_part, e % CS)[rank * per + e / CS] = sum;
      }
      cluster.sync();
      // totals summed over the ranks in rank order
#pragma unroll
      for (int j = 0; j < EPI; ++j) {
        const int q = tid + j * NT;   // q-th element of this rank: e = rank + CS q
        if (q < per) {
          float sum = 0.f;
          for (int r = 0; r < CS; ++r) sum += s_part[r * per + q];
          const int e = rank + CS * q;
          bwd_epilogue(p, L, tile_row0 + e / BP, bp0 + e % BP, sum, pre[j]);
        }
      }
      // no rank reads another one's memory after the barrier above: a rank may leave on its own; before
      // another pass, though, everybody must have read the slices this pass delivered
      if (bp0 + BP < p.B) cluster.sync();
    }
  }
}

// ------------------------------------------------------------------------------------------
// Event-driven backward step for a pseudo-derivative with compact support (SNN_SURR_TRIANGLE, LIF cell).
//
// sigma'(V - theta) = beta max(0, 1 - beta |V - theta|) is exactly zero unless the membrane is within 1 / beta of
// the threshold, and then delta_t = alpha delta_{t+1} needs no product at all.  Only for the near-threshold
// (sample, neuron) pairs are row i of W_rec (and of W_ff of the layer above) multiplied with the deltas: the
// backward pass reads the rows the activity selects, like the forward pass, instead of streaming every matrix
// every step.  A warp owns 32 adjacent neurons of one sample and finds the near-threshold ones by ballot; the
// eight warps of a CTA then share out the CTA's near-threshold neurons in turn and compute their dot products,
// the 32 lanes striding over the contraction index (16-byte
// loads; four accumulators per lane combined in a fixed order, then a fixed shuffle tree: the sum does not depend
// on how the sequence is cut).  Launched as a layer wavefront like bwd_step_kernel (blockIdx.z = layer).
constexpr int BEV_WARPS = 8;

__device__ __forceinline__ float warp_dot(const float* __restrict__ w, const float* __restrict__ d, int n, int lane) {
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  int k = lane * 4;   // n is a multiple of 4
  // eight 16-byte pieces of each operand in flight per lane; the order of the additions is that of the plain loop
  for (; k + 7 * 128 < n; k += 8 * 128) {
    float4 x[8], y[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      x[u] = ldg4_stream(w + k + u * 128);
      y[u] = __ldcg(reinterpret_cast<const float4*>(d + k + u * 128));
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      a0 = fmaf(x[u].x, y[u].x, a0); a1 = fmaf(x[u].y, y[u].y, a1);
      a2 = fmaf(x[u].z, y[u].z, a2); a3 = fmaf(x[u].w, y[u].w, a3);
    }
  }
  for (; k < n; k += 128) {
    const float4 x = ldg4_stream(w + k);
    const float4 y = __ldcg(reinterpret_cast<const float4*>(d + k));
    a0 = fmaf(x.x, y.x, a0); a1 = fmaf(x.y, y.y, a1); a2 = fmaf(x.z, y.z, a2); a3 = fmaf(x.w, y.w, a3);
  }
  float a = (a0 + a1) + (a2 + a3);
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) a += __shfl_xor_sync(0xffffffffu, a, s);
  return a;
}

__global__ void __launch_bounds__(32 * BEV_WARPS) bwd_event_kernel(const __grid_constant__ BwdParams p) {
  pdl_launch_dependents();
  const BwdLayer& L = p.lay[blockIdx.z];
  if (L.mode == 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int strips = (L.N + 31) / 32;   // per sample
  const long long n_strips = (long long)strips * p.B, strip0 = (long long)blockIdx.x * BEV_WARPS;
  if (strip0 >= n_strips) return;       // the whole CTA
  __shared__ uint32_t s_near[BEV_WARPS];
  __shared__ float s_sum[BEV_WARPS * 32];
  const long long strip = strip0 + warp;
  const bool live = strip < n_strips;
  const int b = live ? (int)(strip / strips) : 0, i = live ? (int)(strip % strips) * 32 + lane : 0;
  const bool ok = live && i < L.N;
  pdl_wait();
  const size_t k = (size_t)b * L.N + (ok ? i : 0);
  const float v = ok ? L.V_delta[k] : 0.f;
  const float dn = ok ? __ldcg(L.d_next + k) : 0.f;
  const float u = fmaf(-p.beta, fabsf(v - p.theta), 1.f);
  const float sp = ok && u > 0.f ? p.beta * u : 0.f;   // the same expression as surrogate_grad
  const uint32_t near = __ballot_sync(0xffffffffu, sp != 0.f);
  if (lane == 0) s_near[warp] = near;
  __syncthreads();
  // the near-threshold neurons of the CTA's strips, dealt out to its warps in turn (a strip may hold several)
  int e = 0;
  for (int ws = 0; ws < BEV_WARPS; ++ws) {
    uint32_t bits = s_near[ws];
    while (bits) {
      const int j = __ffs(bits) - 1;
      bits &= bits - 1;
      if (e++ % BEV_WARPS != warp) continue;
      const long long st = strip0 + ws;
      const int bb = (int)(st / strips), row = (int)(st % strips) * 32 + j;
      float sum = 0.f;
      if (L.W_ffa) sum = warp_dot(L.W_ffa + (size_t)row * L.N_post, L.d_above + (size_t)bb * L.N_post, L.N_post, lane);
      sum += warp_dot(L.W_rec + (size_t)row * L.N, L.d_next + (size_t)bb * L.N, L.N, lane);
      if (lane == 0) s_sum[ws * 32 + j] = sum;
    }
  }
  __syncthreads();
  if (ok) {
    float dl = p.alpha * dn;
    if (sp != 0.f) {
      float g = s_sum[warp * 32 + lane] + (L.g_out ? L.g_out[k] : 0.f);
      g = fmaf(-p.theta, dn, g);
      dl = fmaf(g, sp, dl);
    }
    L.V_delta[k] = dl;
    if (L.carry_out) L.carry_out[k] = dl;
  }
}

// ------------------------------------------------------------------------------------------
// Backward steps of ONE layer over a run of steps in one cooperative launch, the recurrent matrix streaming
// from HBM without a pause (networks whose weights exceed L2: the layer-by-layer order).
//
// With one launch per step the HBM stream of W_rec stops at every step boundary: the next launch cannot start
// its copies before delta_t is complete.  But the weights do not depend on the step.  Here a CTA (32 rows of
// W_rec, all samples, the whole contraction range: no cluster) walks through the steps itself and its copy ring
// never drains: while the last chunks of step t are multiplied, the W tiles of the first chunks of step t-1 are
// already on their way; only their delta tiles wait until every CTA has published its rows of delta_t (one counter
// of finished (CTA, step) pairs, release add / acquire poll).
//
// Roles.  Two producer threads issue tiled bulk copies (TMA) into a ring of stages: per chunk of 128 contraction
// values one issues the W tile [32 rows][128] and the other the delta tile [BP samples][128], each as four boxes
// of 32 values (128 bytes per row, 128-byte swizzle: the fragment loads below are then spread over the banks).  A
// stage's `full` barrier takes two arrivals, one that announces the bytes of the W tile and one for the delta tile,
// so the two halves are issued at different times: the W side runs ahead across a step boundary, the delta side
// waits there for the other CTAs.  NWARP consumer warps wait for `full`, multiply their own k-steps of the
// chunk (3-pass TF32 on mma.sync, fragments read straight from the swizzled stage), and arrive on the stage's
// `empty` barrier.  The consumers execute no copy instruction and no address arithmetic for copies.
// Tiling, arithmetic and order of additions are those of bwd_step_kernel with a cluster of one: bit-identical
// results.  Parts of a box outside the matrix arrive as zeros.  When N is a multiple of 32 the tensor maps see the
// contraction index as [N / 32][32] and a tile is one copy instead of four (the producers' trips round their loops
// bound the launch, above all with tiles of 16 rows).  Cooperative launch (all CTAs resident); every
// wait is bounded, and a wait that runs out raises STATUS_SYNC_TIMEOUT: a producer stops issuing, tells the
// consumers and waits for its copies to land (the other producer's next wait then runs out too); a consumer warp stops waiting and computing but keeps taking part in the
// CTA's barriers until the launch ends.
struct BwdStreamParams {
  CUtensorMap map_w;        // W_rec [N][N], box 32 rows x 32 values, 128-byte swizzle
  CUtensorMap map_d;        // delta slots of the run [ts_hi][B][N] (slot buf_slot + z at z), box 1 x BP x 32
  CUtensorMap map_d0;       // delta_{t+1} of the run's latest step [1][B][N], same box
  const float* g_out;       // [B][N] (last layer) or null
  const float* g_ff;        // feed-forward term of the run [n_steps][B][N] (first row: step t0 + ts_lo + 1), or null;
                            // g_ff_parts partial sums over slices of the contraction range, g_ff_stride floats apart
  size_t g_ff_stride;
  int g_ff_parts;
  const float* d_first;     // [B][N] delta_{t+1} of the run's latest step
  float* carry_out;         // [B][N] receives delta of the step with ts == 0, or null
  float* slots;             // state slot s starts at slots + s * slot_stride
  size_t slot_stride;       // floats
  size_t state_off;         // offset of this layer inside a state slot, in floats
  uint32_t* status;
  uint32_t* progress;       // finished (CTA, step) pairs, zero at launch
  int N, B;
  int buf_slot, ts_lo, ts_hi;   // steps ts = ts_hi-1 .. ts_lo; slot buf_slot + ts holds V on entry, delta on exit
  int keep_chunks;              // the first keep_chunks chunks of 128 contraction values are asked to stay in L2
  int one_copy;                 // N is a multiple of 32: the maps see the contraction index as [N / 32][32] and a tile is ONE
                                // copy (map_w [N / 32][N rows][32], box 4 x 16 MT x 32; map_d, map_d0 [slots][N / 32][B][32])
  float alpha, theta, beta;
  int surrogate, cell;
};

constexpr size_t BWD_STREAM_KEEP_BYTES = (size_t)64 << 20;   // of W_rec kept in L2 across the steps of a run

// stages of the ring: what fits beside the partial tiles with two CTAs per SM (one for the 16-warp instance)
template <int NTN, int MT> __host__ __device__ constexpr int bwd_stream_stages() {
  return MT == 2 ? (NTN == 2 ? 3 : 4) : (NTN == 2 ? 5 : 6);
}

// MT = tiles of 16 rows per CTA: 2 where that still gives every SM a CTA, else 1 (twice the CTAs for layers half as wide)
template <int NTN, int NWARP, int MT>
__host__ __device__ constexpr size_t bwd_stream_smem_bytes() {
  // the ring (stages of a W tile and a delta tile), the warps' partial tiles, and room to align the ring to 1024 bytes
  return (size_t)bwd_stream_stages<NTN, MT>() * (16 * MT + 8 * NTN) * 128 * sizeof(float) +
         (size_t)NWARP * 16 * MT * (8 * NTN + 8) * sizeof(float) + 1024;
}

template <int NTN, int NWARP, int MT>
__global__ void __launch_bounds__(32 * (NWARP + 2), NWARP == 8 ? 2 : 1) bwd_stream_kernel(const __grid_constant__ BwdStreamParams p) {
  constexpr int KS = 16 / NWARP, KW = 8 * KS, S = bwd_stream_stages<NTN, MT>();
  constexpr int TM = 16 * MT;                                                         // rows per CTA
  constexpr int NT = 32 * NWARP, BP = 8 * NTN, TILE = TM * BP;
  constexpr int TS = BP + 8, TILEP = TM * TS;
  constexpr int EPI = (TILE + NT - 1) / NT;
  constexpr uint32_t W_BOX_BYTES = TM * 128, D_BOX_BYTES = BP * 128;                  // one box of 32 values
  constexpr uint32_t W_TILE_BYTES = 4 * W_BOX_BYTES, STAGE_BYTES = W_TILE_BYTES + 4 * D_BOX_BYTES;
  static_assert(W_BOX_BYTES % 1024 == 0 && D_BOX_BYTES % 1024 == 0, "every box starts at a multiple of the swizzle period");
  const int tile_row0 = blockIdx.x * TM;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  __shared__ uint64_t s_full[S], s_empty[S];
  __shared__ int s_abort;
  extern __shared__ unsigned char s_dyn_raw[];
  unsigned char* const ring = reinterpret_cast<unsigned char*>(((uintptr_t)s_dyn_raw + 1023) & ~(uintptr_t)1023);
  float* const s_parts = reinterpret_cast<float*>(ring + (size_t)S * STAGE_BYTES);   // [NWARP][32][TS] partial tiles
  const int N = p.N, it_all = (N + 127) / 128, n_steps = p.ts_hi - p.ts_lo;
  const int total = n_steps * it_all;                                 // chunks of the whole run
  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(s_full + s, 2); mbar_init(s_empty + s, NWARP); }
    mbar_fence_init();
    s_abort = 0;
  }
  __syncthreads();

  if (warp >= NWARP) {
    // ---- producers: one thread for the W tiles, one for the delta tiles.  What bounds the launch is how fast such a
    // thread gets round its loop, so the loops hold nothing they can do without (one thread issuing both tiles: 46.7 us
    // per step; two threads: 42.5 us; a look at the abort flag per chunk or both roles in one loop cost 2 to 4 % each).
    // A producer learns that the launch is failing when one of its own waits runs out.
    if (lane != 0) return;
    int st = 0, it = 0;          // stage and index within its step of chunk c
    uint32_t round = 0;          // c / S: chunk c waits for the `empty` phase round - 1 of its stage
    int c = 0;
    bool ok = true;
    if (warp == NWARP) {
      // The matrix is read once per step and is larger than L2, so left to itself every step would fetch all of it
      // from HBM.  The first keep_chunks chunks are fetched with the lowest eviction priority and the others with the
      // highest: that part of the matrix is still in L2 when the next step asks for it.
      const uint64_t pol_keep = l2_keep_policy(), pol_stream = l2_stream_policy();
      for (; c < total; ++c) {
        if (c >= S && !mbar_wait(s_empty + st, (round - 1u) & 1u)) { ok = false; break; }   // chunk c - S is consumed
        uint64_t* const bar = s_full + st;
        unsigned char* const dst = ring + (size_t)st * STAGE_BYTES;
        mbar_arrive_expect_tx(bar, W_TILE_BYTES);
        const uint64_t pol = it < p.keep_chunks ? pol_keep : pol_stream;
        if (p.one_copy) {
          tma_load_3d_hint(dst, &p.map_w, 0, tile_row0, it * 4, bar, pol);
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q) tma_load_2d_hint(dst + q * W_BOX_BYTES, &p.map_w, it * 128 + 32 * q, tile_row0, bar, pol);
        }
        if (++st == S) { st = 0; ++round; }
        if (++it == it_all) it = 0;
      }
    } else {
      int s = 0;                 // step of chunk c
      for (; c < total; ++c) {
        if (c >= S && !mbar_wait(s_empty + st, (round - 1u) & 1u)) { ok = false; break; }
        if (it == 0 && s > 0) {  // first chunk of a step: every CTA has written its rows of delta_{t+1}
          if (!wait_progress(p.progress, (uint32_t)gridDim.x * (uint32_t)s)) { ok = false; break; }
          fence_proxy_async_all();   // the other CTAs' stores, seen through the counter, before the copies that read them
        }
        uint64_t* const bar = s_full + st;
        unsigned char* const dst = ring + (size_t)st * STAGE_BYTES + W_TILE_BYTES;
        mbar_arrive_expect_tx(bar, 4 * D_BOX_BYTES);
        const CUtensorMap* const map = s == 0 ? &p.map_d0 : &p.map_d;
        const int z = s == 0 ? 0 : p.ts_hi - s;
        if (p.one_copy) {
          tma_load_4d(dst, map, 0, 0, it * 4, z, bar);
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q) tma_load_3d(dst + q * D_BOX_BYTES, map, it * 128 + 32 * q, 0, z, bar);
        }
        if (++st == S) { st = 0; ++round; }
        if (++it == it_all) { it = 0; ++s; }
      }
    }
    if (!ok) {
      // give up: raise the status, tell the consumers, and wait (briefly: the copies were issued long ago, and a
      // barrier whose other half was never issued cannot complete) for the stages this thread has copies in
      atomicOr(p.status, STATUS_SYNC_TIMEOUT);
      *reinterpret_cast<volatile int*>(&s_abort) = 1;
      for (int cc = c > S ? c - S : 0; cc < c; ++cc) mbar_wait(s_full + cc % S, (uint32_t)(cc / S) & 1u, 1u << 14);
    }
    return;
  }

  // ---- consumers
  // this lane's fragment position inside a box: row g, values k_lane .. of the chunk (k_lane = KW warp + 2 KS t),
  // i.e. box k_lane / 32, 16-byte piece (k_lane % 32) / 4 exchanged with piece ^ (row % 8) by the swizzle
  const int k_lane = KW * warp + 2 * KS * t;
  const int frag = g * 32 + ((((k_lane & 31) >> 2) ^ g) << 2) + (k_lane & 3);   // floats; rows g + 8 r share row % 8
  const int w_off = (k_lane >> 5) * (W_BOX_BYTES / 4) + frag, d_off = (int)(W_TILE_BYTES / 4) + (k_lane >> 5) * (D_BOX_BYTES / 4) + frag;
  auto consumer_barrier = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(NT) : "memory"); };
  // delta_{t+1} of the s-th step of the run (s = 0: the latest)
  auto dn_of = [&](int s) -> const float* {
    return s == 0 ? p.d_first : p.slots + (size_t)(p.buf_slot + p.ts_hi - s) * p.slot_stride + p.state_off;
  };
  bool dead = false;   // a wait of this warp ran out: no more waiting or computing, only the CTA's barriers
  int st = 0;
  uint32_t ph_full = 0;
  for (int s = 0; s < n_steps; ++s) {
    const int ts = p.ts_hi - 1 - s;
    const float* const dn = dn_of(s);
    float* const Vd = p.slots + (size_t)(p.buf_slot + ts) * p.slot_stride + p.state_off;
    const float* const gff = p.g_ff ? p.g_ff + (size_t)(ts - p.ts_lo) * p.B * N : nullptr;
    // what the epilogue needs, fetched now.  The rows of delta_{t+1} read here are this CTA's own (written before
    // the barrier that ended the previous step); the first step's come from before the launch.
    float pre_dn[EPI], pre_go[EPI], pre_gf[EPI], pre_v[EPI];
#pragma unroll
    for (int j = 0; j < EPI; ++j) {
      const int e = tid + j * NT, i = tile_row0 + e / BP, b = e % BP;
      pre_dn[j] = pre_go[j] = pre_gf[j] = pre_v[j] = 0.f;
      if (e < TILE && i < N && b < p.B) {
        const size_t k = (size_t)b * N + i;
        pre_dn[j] = __ldcg(dn + k);
        pre_go[j] = p.g_out ? p.g_out[k] : 0.f;
        if (gff) {   // the partial sums in slice order
          pre_gf[j] = gff[k];
          for (int q = 1; q < p.g_ff_parts; ++q) pre_gf[j] += gff[(size_t)q * p.g_ff_stride + k];
        }
        pre_v[j] = Vd[k];
      }
    }
    float acc[MT][NTN][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
    if (!dead) {
      for (int it = 0; it < it_all; ++it) {
        if (!mbar_wait(s_full + st, ph_full)) {
          if (lane == 0) atomicOr(p.status, STATUS_SYNC_TIMEOUT);
          dead = true;
          break;
        }
        const float* const stage = reinterpret_cast<const float*>(ring + (size_t)st * STAGE_BYTES);
        warp_chunk_mma<NTN, KS, MT>(acc, stage + w_off, 32, stage + d_off, 32, [](int) {});
        __syncwarp();
        if (lane == 0) mbar_arrive(s_empty + st);
        if (++st == S) { st = 0; ph_full ^= 1u; }
      }
    }
    // the warps' partial tiles, summed in warp order
    {
      float* mine = s_parts + (size_t)warp * TILEP;
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt) {
          const int r = mt * 16 + g, cc = nt * 8 + 2 * t;
          *reinterpret_cast<float2*>(mine + r * TS + cc) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
          *reinterpret_cast<float2*>(mine + (r + 8) * TS + cc) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
    }
    consumer_barrier();
    if (s_abort) dead = true;
#pragma unroll
    for (int j = 0; j < EPI; ++j) {
      const int e = tid + j * NT, i = tile_row0 + e / BP, b = e % BP;
      float sum = 0.f;
      if (e < TILE) {
#pragma unroll
        for (int w = 0; w < NWARP; ++w) sum += s_parts[(size_t)w * TILEP + (e / BP) * TS + e % BP];
      }
      if (e < TILE && i < N && b < p.B && !dead) {
        const size_t k = (size_t)b * N + i;
        float gs = sum + pre_go[j];
        if (gff) gs += pre_gf[j];
        if (p.cell == 0) gs = fmaf(-p.theta, pre_dn[j], gs);
        const float sp = surrogate_grad(pre_v[j], p.theta, p.beta, p.surrogate, p.cell);
        const float dl = fmaf(gs, sp, p.alpha * pre_dn[j]);
        Vd[k] = dl;
        if (ts == 0 && p.carry_out) p.carry_out[k] = dl;
      }
    }
    fence_proxy_async_all();   // these stores before the other CTAs' bulk copies that the counter lets go
    consumer_barrier();        // delta_t of this CTA is written, and the partial tiles are free again
    if (tid == 0) publish_progress(p.progress);
  }
}

// ------------------------------------------------------------------------------------------
// Backward pass over a whole segment in one cooperative launch, the weights resident in shared memory
// (networks small enough that a CTA's slice of both matrices, 32 rows x its share of the contraction
// index, fits beside the staging ring).
//
// Same tiling, same arithmetic and the same order of additions as bwd_step_kernel (results are
// bit-identical), but a CTA loads its slice of W_ff(l+1) and W_rec once and then walks through the steps
// t1 .. t0+1 itself; per step only delta streams in, every warp staging the values of its own k-steps
// in a cp.async ring of its own (no barrier between warps inside the contraction).  Layer l may start step t
// when all of delta^l_{t+1} and delta^{l+1}_t is written: one counter of finished (CTA, step) pairs per
// layer, published with a release add after a CTA barrier, polled with acquire loads; delta is then
// read past L1.  The slices a rank receives from the other ranks of its cluster alternate between two
// buffers, so a rank that is one step ahead never overwrites what a slower one still reads.  A wait
// that runs out raises STATUS_SYNC_TIMEOUT; the CTA then stops waiting but keeps taking part in every
// barrier until the end of the launch (a CTA that left early would block its cluster).
struct BwdSegLayer {
  const float* W_rec;       // [N][N]
  const float* W_ffa;       // W_ff of the layer above [N][N_post] or null
  const float* g_out;       // [B][N] (last layer) or null
  const float* carry_in;    // [B][N] delta^l_{t1+1}
  float* carry_out;         // [B][N] receives delta^l_{t0+1}
  size_t state_off;         // offset of this layer inside a state slot, in floats
  size_t state_off_above;   // of the layer above
  int N, N_post;
  int ctas;                 // CTAs of this layer (row tiles x cluster size)
  int cta0;                 // blockIdx.x of its first CTA (a multiple of the cluster size)
};

struct BwdSegParams {
  BwdSegLayer lay[MAXL];
  float* slots;
  size_t slot_stride;       // floats
  uint32_t* status;
  uint32_t* progress;       // [L] finished (CTA, step) pairs per layer, zero at launch
  int L, B, t0, t1, buf_slot;   // step t lives in slot buf_slot + (t - t0 - 1): V_t on entry, delta_t on exit
  float alpha, theta, beta;
  int surrogate, cell;
};

constexpr int BSEG_STAGES = 3;   // chunks of delta in flight per warp

// floats of the resident slice per row: every chunk of 128 k (feed-forward part first, each part padded to
// whole chunks with zeros) plus the padding that makes the lanes' vector loads conflict-free (bwd_ld)
__host__ __device__ inline int bwd_resident_ld(int k_ff, int k_rec, int nwarp) {
  return ((k_ff + 127) / 128 + (k_rec + 127) / 128) * 128 + (bwd_ld(nwarp) - 128);
}
template <int NTN, int NWARP> __host__ __device__ constexpr size_t bwd_segment_region_floats() {
  // the warps' delta rings (per stage the warp's 8 KS values of a chunk for BP samples: 128 BP floats over all
  // warps), reused for their partial tiles
  return (size_t)(BSEG_STAGES * 128 * 8 * NTN) > (size_t)(NWARP * BWD_TM * (8 * NTN + 8))
             ? (size_t)(BSEG_STAGES * 128 * 8 * NTN) : (size_t)(NWARP * BWD_TM * (8 * NTN + 8));
}

template <int NTN, int NWARP>
__global__ void __launch_bounds__(32 * NWARP, 1) bwd_segment_kernel(const __grid_constant__ BwdSegParams p) {
  constexpr int NT = 32 * NWARP, BP = 8 * NTN, TILE = BWD_TM * BP;
  constexpr int TS = BP + 8, TILEP = BWD_TM * TS;
  constexpr int EPI = TILE / NT;
  constexpr int KS = 16 / NWARP;                 // k-steps of a chunk per warp
  constexpr int KW = 8 * KS;                     // its contraction values per chunk, adjacent
  constexpr int WSTAGE_F = BP * KW;              // floats of one warp's stage: BP samples x KW values
  constexpr int PIECES = BP * KW / 4;            // 16-byte pieces of it
  constexpr int ITER = (PIECES + 31) / 32;       // per lane
  static_assert(TILE % NT == 0 && 16 % NWARP == 0, "tiles divide evenly among the threads");
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  int l = 0;
  while (l + 1 < p.L && (int)blockIdx.x >= p.lay[l + 1].cta0) ++l;
  const BwdSegLayer& L = p.lay[l];
  const int tile_row0 = (((int)blockIdx.x - L.cta0) / CS) * BWD_TM;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
  const bool above = L.W_ffa != nullptr;
  __shared__ float s_part[2][TILE];
  __shared__ int s_ok, s_dead;
  extern __shared__ float4 s_dyn[];
  // this rank's slice of each contraction range, in units of 4 floats
  const int q_rec = L.N / 4, q_ff = above ? L.N_post / 4 : 0;
  const int lo_rec = (int)((long long)q_rec * rank / CS) * 4, hi_rec = (int)((long long)q_rec * (rank + 1) / CS) * 4;
  const int lo_ff = (int)((long long)q_ff * rank / CS) * 4, hi_ff = (int)((long long)q_ff * (rank + 1) / CS) * 4;
  const int it_ff = (hi_ff - lo_ff + 127) / 128, it_all = it_ff + (hi_rec - lo_rec + 127) / 128;
  const int LDW = it_all * 128 + (bwd_ld(NWARP) - 128);
  float* const Wres = reinterpret_cast<float*>(s_dyn);             // [32][LDW]
  float* const s_reg = Wres + (size_t)BWD_TM * LDW;                // per-warp delta rings [NWARP][BSEG_STAGES][BP][KW]; later partial tiles
  float* const ring = s_reg + (size_t)warp * BSEG_STAGES * WSTAGE_F;
  const int rlast = L.N - 1, blast = p.B - 1;

  // ---- the resident slice: rows tile_row0 .. +31, chunk by chunk, zeros past a part's end and past row N-1
  for (int q = tid; q < BWD_TM * it_all * 32; q += NT) {
    const int rr = q / (it_all * 32), c4 = q % (it_all * 32), it = c4 >> 5, kc = (c4 & 31) * 4;
    const bool ff = it < it_ff;
    const int k = ff ? lo_ff + it * 128 + kc : lo_rec + (it - it_ff) * 128 + kc;
    const bool real = tile_row0 + rr <= rlast && k < (ff ? hi_ff : hi_rec);
    const float* src = ff ? L.W_ffa + (size_t)(tile_row0 + rr) * L.N_post + k : L.W_rec + (size_t)(tile_row0 + rr) * L.N + k;
    cp_async16_or_zero(Wres + (size_t)rr * LDW + c4 * 4, real ? src : L.W_rec, real);
  }
  cp_async_commit();
  if (tid == 0) s_dead = 0;
  cp_async_wait<0>();
  __syncthreads();

  uint32_t* const my_progress = p.progress + l;
  const int n_steps = p.t1 - p.t0;
  for (int d = 1; d <= n_steps; ++d) {
    const int t = p.t1 - d + 1;
    if (tid == 0) {
      bool ok = s_dead == 0;
      if (ok) ok = wait_progress(my_progress, (uint32_t)L.ctas * (uint32_t)(d - 1));
      if (ok && above) ok = wait_progress(p.progress + (l + 1), (uint32_t)p.lay[l + 1].ctas * (uint32_t)d);
      if (!ok && s_dead == 0) { atomicOr(p.status, STATUS_SYNC_TIMEOUT); s_dead = 1; }
      s_ok = ok ? 1 : 0;
    }
    __syncthreads();
    const bool live = s_ok != 0;   // after a timeout the CTA only keeps the barriers going
    float* const Vd = p.slots + (size_t)(p.buf_slot + (t - p.t0 - 1)) * p.slot_stride + L.state_off;
    const float* const dn = d == 1 ? L.carry_in
                                   : p.slots + (size_t)(p.buf_slot + (t - p.t0)) * p.slot_stride + L.state_off;
    const float* const da = above ? p.slots + (size_t)(p.buf_slot + (t - p.t0 - 1)) * p.slot_stride + L.state_off_above
                                  : nullptr;
    float* const part = s_part[d & 1];

    for (int bp0 = 0; bp0 < p.B; bp0 += BP) {
      // what the epilogue needs, fetched now (delta_{t+1} was written by other CTAs of this launch: past L1)
      float pre_dn[EPI], pre_go[EPI], pre_v[EPI];
#pragma unroll
      for (int j = 0; j < EPI; ++j) {
        const int q = tid + j * NT, e = CS == 1 ? q : rank + CS * q;
        const int i = tile_row0 + e / BP, b = bp0 + e % BP;
        pre_dn[j] = pre_go[j] = pre_v[j] = 0.f;
        if (live && e < TILE && i < L.N && b < p.B) {
          const size_t k = (size_t)b * L.N + i;
          pre_dn[j] = __ldcg(dn + k);
          pre_go[j] = L.g_out ? L.g_out[k] : 0.f;
          pre_v[j] = Vd[k];
        }
      }
      // Every warp stages the delta values of its own k-steps (KW adjacent values x BP samples: KW / 4 16-byte
      // pieces per sample) in a ring of its own, so that no warp waits for another one inside the contraction and the
      // loads, splits and tensor-core passes of different warps overlap.  A lane copies fixed pieces.
      const float* src_rec[ITER];
      const float* src_ff[ITER];
      int dst_off[ITER], kofs[ITER];
#pragma unroll
      for (int j = 0; j < ITER; ++j) {
        const int q = lane + j * 32;                                   // piece: (sample, quarter of the warp's values)
        const int sm = q / (KW / 4), part = q % (KW / 4);
        kofs[j] = q < PIECES ? warp * KW + part * 4 : -1;              // k inside the chunk
        dst_off[j] = sm * KW + part * 4;
        const size_t b = bp0 + sm < blast ? bp0 + sm : blast;           // samples past the batch: a valid row, never used
        src_rec[j] = dn + b * L.N;
        src_ff[j] = above ? da + b * L.N_post : nullptr;
      }
      auto issue = [&](int it) {
        if (it < it_all) {
          const bool ff = it < it_ff;
          const int k0 = ff ? lo_ff + it * 128 : lo_rec + (it - it_ff) * 128;
          const int hi = ff ? hi_ff : hi_rec;
          float* st = ring + (size_t)(it % BSEG_STAGES) * WSTAGE_F;
#pragma unroll
          for (int j = 0; j < ITER; ++j) {
            if (kofs[j] < 0) continue;
            const int k = k0 + kofs[j];
            cp_async16_or_zero(st + dst_off[j], k < hi ? (ff ? src_ff[j] : src_rec[j]) + k : L.W_rec, k < hi);
          }
        }
        cp_async_commit();
      };
      float acc[2][NTN][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
      for (int it = 0; it < BSEG_STAGES - 1; ++it) issue(it);
      for (int it = 0; it < it_all; ++it) {
        cp_async_wait<BSEG_STAGES - 2>();   // this lane's pieces of chunk `it` have landed
        __syncwarp();                       // ... the whole warp's have, and the warp is done with chunk it-1
        issue(it + BSEG_STAGES - 1);        // refills the stage chunk it-1 used
        const float* Wc = Wres + it * 128;
        const float* Ds = ring + (size_t)(it % BSEG_STAGES) * WSTAGE_F;
        warp_chunk_mma<NTN, KS>(acc, Wc + (size_t)g * LDW + warp * KW + 2 * KS * t4, LDW, Ds + g * KW + 2 * KS * t4, KW,
                                [](int) {});
      }
      cp_async_wait<0>();
      __syncthreads();   // the ring is free: it now holds the warps' partial tiles [NWARP][32][TS]
      {
        float* mine = s_reg + (size_t)warp * TILEP;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int nt = 0; nt < NTN; ++nt) {
            const int r = mt * 16 + g, c = nt * 8 + 2 * t4;
            *reinterpret_cast<float2*>(mine + r * TS + c) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2*>(mine + (r + 8) * TS + c) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
          }
      }
      __syncthreads();
      auto finish = [&](int e, float sum, int j) {
        const int i = tile_row0 + e / BP, b = bp0 + e % BP;
        if (!live || i >= L.N || b >= p.B) return;
        const size_t k = (size_t)b * L.N + i;
        float gsum = sum + pre_go[j];
        if (p.cell == 0) gsum = fmaf(-p.theta, pre_dn[j], gsum);
        const float sp = surrogate_grad(pre_v[j], p.theta, p.beta, p.surrogate, p.cell);
        const float dl = fmaf(gsum, sp, p.alpha * pre_dn[j]);
        Vd[k] = dl;
        if (t == p.t0 + 1) L.carry_out[k] = dl;
      };
      if (CS == 1) {
#pragma unroll
        for (int j = 0; j < EPI; ++j) {
          const int e = tid + j * NT;
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < NWARP; ++w) sum += s_reg[(size_t)w * TILEP + (e / BP) * TS + e % BP];
          finish(e, sum, j);
        }
        __syncthreads();   // before the ring is refilled
      } else {
        const int per = TILE / CS;
        for (int e = tid; e < TILE; e += NT) {
          float sum = 0.f;
#pragma unroll
          for (int w = 0; w < NWARP; ++w) sum += s_reg[(size_t)w * TILEP + (e / BP) * TS + e % BP];
          cluster.map_shared_rank(part, e % CS)[rank * per + e / CS] = sum;
        }
        cluster.sync();   // also a CTA barrier: the ring may be refilled after it
#pragma unroll
        for (int j = 0; j < EPI; ++j) {
          const int q = tid + j * NT;
          if (q < per) {
            float sum = 0.f;
            for (int r = 0; r < CS; ++r) sum += part[r * per + q];
            finish(rank + CS * q, sum, j);
          }
        }
        if (bp0 + BP < p.B) cluster.sync();   // another pass of this step reuses the same buffer
      }
    }
    __syncthreads();
    if (tid == 0 && live) publish_progress(my_progress);   // this CTA's share of delta_t is written
  }
}

// ------------------------------------------------------------------------------------------
// Time-batched feed-forward part of the backward pass: for a run of steps the deltas of the layer
// above are all known before the layer below starts, so W_ff^{l+1} delta^{l+1}_t is one product
// with M = steps x B columns instead of one per step:
//   out[(ts, b)][i] = sum_k W[i][k] * delta_{t0+1+ts}[b][k]
// W is then streamed once per 64 (step, sample) pairs instead of once per step.  Same machinery as
// bwd_step_kernel: 32 rows of W per CTA, 128-wide chunks of k through a cp.async pipeline, 3-pass
// TF32 tensor-core product, warp partials summed in warp order; per output the order of additions
// depends on k only, not on which pairs share a tile.
struct FfGemmParams {
  const float* W;        // [N][K]   W_ff of the layer above (row = neuron of this layer)
  const float* delta0;   // delta of the layer above at the first step of the run: row (ts, b) at
                         //   delta0 + ts * slot_stride + b * K
  float* out;            // [n_steps * B][N]
  size_t slot_stride;    // floats between consecutive steps
  int N, K, B, n_steps;
};

constexpr int FFG_NTN = 8, FFG_NWARP = 16;   // 64 (step, sample) pairs per pass, 16 warps

__global__ void __launch_bounds__(32 * FFG_NWARP, 1) ff_gemm_kernel(const __grid_constant__ FfGemmParams p) {
  constexpr int NTN = FFG_NTN, NWARP = FFG_NWARP, NT = 32 * NWARP, BP = 8 * NTN, ROWS = BWD_TM + BP;
  constexpr int STAGE_F = ROWS * BWD_LD, TILE = BWD_TM * BP, ITER = ROWS * 32 / NT;
  constexpr int BPP = BP + 1, TILEP = BWD_TM * BPP;   // partial tiles padded: conflict-free column reads
  static_assert(ROWS * 32 % NT == 0, "the staged tile divides evenly among the threads");
  pdl_launch_dependents();
  const int tile_row0 = blockIdx.y * BWD_TM;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  extern __shared__ float4 s_dyn[];
  float* const s_tiles = reinterpret_cast<float*>(s_dyn);   // [BWD_STAGES][ROWS][BWD_LD]; later [NWARP][32][BP]
  const int M = p.n_steps * p.B, it_all = (p.K + 127) / 128;
  const int rlast = p.N - 1;
  pdl_wait();
  {   // one pass of 64 (step, sample) pairs per CTA: blockIdx.x selects it, so that the CTAs that read the
      // same rows of W run at the same time and all but the first find them in L2
    const int bp0 = blockIdx.x * BP;
    const float* src[ITER];
    int dst_off[ITER], kcol[ITER];
#pragma unroll
    for (int j = 0; j < ITER; ++j) {
      const int q = tid + j * NT, rr = q >> 5, c4 = q & 31;
      kcol[j] = 4 * c4;
      dst_off[j] = rr * BWD_LD + 4 * c4;
      if (rr < BWD_TM) {   // rows and pairs past the end are clamped to the last valid one; never stored
        const size_t row = tile_row0 + rr < rlast ? tile_row0 + rr : rlast;
        src[j] = p.W + row * p.K + 4 * c4;
      } else {
        const int m = bp0 + rr - BWD_TM < M - 1 ? bp0 + rr - BWD_TM : M - 1;
        src[j] = p.delta0 + (size_t)(m / p.B) * p.slot_stride + (size_t)(m % p.B) * p.K + 4 * c4;
      }
    }
    auto issue = [&](int it) {
      if (it < it_all) {
        const int k0 = it * 128;
        float* st = s_tiles + (size_t)(it % BWD_STAGES) * STAGE_F;
#pragma unroll
        for (int j = 0; j < ITER; ++j) {
          if (k0 + kcol[j] < p.K) cp_async16(st + dst_off[j], src[j] + k0);
          else *reinterpret_cast<float4*>(st + dst_off[j]) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
      cp_async_commit();
    };
    float acc[2][NTN][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NTN; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
    for (int it = 0; it < BWD_STAGES - 1; ++it) issue(it);
    for (int it = 0; it < it_all; ++it) {
      cp_async_wait<BWD_STAGES - 2>();
      __syncthreads();
      issue(it + BWD_STAGES - 1);
      const float* Ws = s_tiles + (size_t)(it % BWD_STAGES) * STAGE_F;
      const float* Ds = Ws + BWD_TM * BWD_LD;
#pragma unroll 1
      for (int ks = warp; ks < 16; ks += NWARP) {
        const int kk = ks * 8 + t;
        uint32_t a_hi[2][4], a_lo[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const float* r0 = Ws + (mt * 16 + g) * BWD_LD + kk;
          split_tf32(r0[0], a_hi[mt][0], a_lo[mt][0]);
          split_tf32(r0[8 * BWD_LD], a_hi[mt][1], a_lo[mt][1]);
          split_tf32(r0[4], a_hi[mt][2], a_lo[mt][2]);
          split_tf32(r0[8 * BWD_LD + 4], a_hi[mt][3], a_lo[mt][3]);
        }
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt) {
          uint32_t b_hi[2], b_lo[2];
          const float* r0 = Ds + (nt * 8 + g) * BWD_LD + kk;
          split_tf32(r0[0], b_hi[0], b_lo[0]);
          split_tf32(r0[4], b_hi[1], b_lo[1]);
          mma_tf32(acc[0][nt], a_lo[0], b_hi); mma_tf32(acc[1][nt], a_lo[1], b_hi);
          mma_tf32(acc[0][nt], a_hi[0], b_lo); mma_tf32(acc[1][nt], a_hi[1], b_lo);
          mma_tf32(acc[0][nt], a_hi[0], b_hi); mma_tf32(acc[1][nt], a_hi[1], b_hi);
        }
      }
    }
    cp_async_wait<0>();
    __syncthreads();   // the stages are free: they now hold the warps' partial tiles [NWARP][32][BP]
    {
      float* mine = s_tiles + (size_t)warp * TILEP;
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTN; ++nt) {
          const int r = mt * 16 + g, c = nt * 8 + 2 * t;
          mine[r * BPP + c] = acc[mt][nt][0];       mine[r * BPP + c + 1] = acc[mt][nt][1];
          mine[(r + 8) * BPP + c] = acc[mt][nt][2]; mine[(r + 8) * BPP + c + 1] = acc[mt][nt][3];
        }
    }
    __syncthreads();
    // out[m][i]: consecutive threads take consecutive rows i of one pair m (coalesced stores)
    for (int e = tid; e < TILE; e += NT) {
      const int r = e % BWD_TM, c = e / BWD_TM;
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < NWARP; ++w) sum += s_tiles[(size_t)w * TILEP + r * BPP + c];
      const int i = tile_row0 + r, m = bp0 + c;
      if (i < p.N && m < M) p.out[(size_t)m * p.N + i] = sum;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Sparse outer-product weight gradient over a run of steps t = t1 .. t0+1:
//   dW[j, :] += delta_t[b, :]   for every (t, b) in which presynaptic neuron j was active,
// accumulated per element in the fixed order t descending, b ascending, starting from the
// value already in dW.  A CTA owns 8 presynaptic rows (one warp each) and a column tile.
// The (t, b) pairs are scanned in windows of DW_WINDOW: the warps first compact, by ballot
// over the spike words, the list of pairs in which their row was active, then stream the
// listed delta rows with DW_BATCH loads in flight, adding them in list order.
struct DwArgs {
  float* dW;                 // [N_pre][N]
  const uint32_t* mask_row0; // spike words of the presynaptic layer for t = t0+1: [(t-t0-1)][B][Wm]
  const float* delta0;       // delta of step t0+1: delta(t, b) = delta0 + (t-t0-1) * slot_stride + b * N
  int N_pre, N, Wm;
  // graded cell only: where the value of an event is found (same step indexing as mask_row0)
  const uint32_t* off_row0;  // list offsets of the presynaptic layer [(t-t0-1)][B]
  const uint16_t* pref_row0; // events before each spike word [(t-t0-1)][B][Wm]
  const float* vals;         // value pool [B][cap]
  size_t cap;
};

// All weight matrices of a segment in one launch: blockIdx.z selects the matrix.
struct DwParams {
  DwArgs m[2 * MAXL];
  size_t slot_stride;        // floats between consecutive steps (multiple of 4)
  int B, n_steps;
  int window;                // (t, b) pairs compacted at a time: min(n_steps * B rounded up to 32, DW_WINDOW)
  int slab_rows;             // dw_slab_kernel: presynaptic rows per CTA
};

constexpr int DW_ROWS = 8;        // rows (warps) per CTA
constexpr int DW_WINDOW = 1024;   // (t, b) pairs compacted at a time
// delta rows per copy group: 4, 2 or 1 as the column tile widens (keeps the ring at 64 KB per CTA)
template <int U> __host__ __device__ constexpr int dw_group() { return U >= 8 ? 1 : U >= 4 ? 2 : 4; }
constexpr int DW_STAGES = 2;      // copy groups in flight per warp

// shared memory of dw_kernel in bytes for a window of `window` pairs
template <int U, bool GRADED> constexpr size_t dw_smem_bytes(int window) {
  return (size_t)DW_ROWS * DW_STAGES * dw_group<U>() * U * 32 * sizeof(float4) +
         (size_t)window * sizeof(uint32_t) * (2 + DW_ROWS + (GRADED ? 1 + DW_ROWS : 0));
}

template <int U, bool GRADED>
__global__ void __launch_bounds__(32 * DW_ROWS) dw_kernel(const __grid_constant__ DwParams p) {
  constexpr int DW_GROUP = dw_group<U>();
  pdl_launch_dependents();
  const DwArgs& a = p.m[blockIdx.z];
  if ((int)blockIdx.y * DW_ROWS >= a.N_pre || (int)blockIdx.x * 128 * U >= a.N) return;
  pdl_wait();
  // dynamic shared memory: copy ring [DW_ROWS][DW_STAGES][DW_GROUP][U][32] float4; then, per window,
  // the spike words [window], the position of each pair's delta row in units of 16 bytes [window],
  // and per row the list of those positions for the pairs in which the row fired [DW_ROWS][window];
  // graded cell: also each pair's (step, sample) row index and per row the event values
  extern __shared__ float4 s_ring[];
  const int window = p.window, B = p.B, n_steps = p.n_steps;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t* const s_words = reinterpret_cast<uint32_t*>(s_ring + (size_t)DW_ROWS * DW_STAGES * DW_GROUP * U * 32);
  uint32_t* const s_off = s_words + window;
  uint32_t* const s_evw = s_off + window + (size_t)warp * window;
  uint32_t* const s_rowi = s_off + (size_t)(1 + DW_ROWS) * window;            // graded only
  float* const s_valw = reinterpret_cast<float*>(s_rowi + window) + (size_t)warp * window;
  const int row = blockIdx.y * DW_ROWS + warp;
  const int wc = (blockIdx.y * DW_ROWS) >> 5;               // spike word column of these rows
  const int bit = ((blockIdx.y * DW_ROWS) & 31) + warp;     // this row's bit in it
  const int colb = blockIdx.x * (128 * U) + lane * 4;
  const bool row_ok = row < a.N_pre;
  float4 acc[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    const int c = colb + u * 128;
    acc[u] = (row_ok && c < a.N) ? *reinterpret_cast<const float4*>(a.dW + (size_t)row * a.N + c)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float4* const ring = s_ring + (size_t)warp * DW_STAGES * DW_GROUP * U * 32 + lane;
  const float4* const delta_c = reinterpret_cast<const float4*>(a.delta0 + colb);
  const uint32_t stride16 = (uint32_t)(p.slot_stride / 4), n16 = (uint32_t)(a.N / 4);
  const int n_pairs = n_steps * B;
  for (int p0 = 0; p0 < n_pairs; p0 += window) {
    const int lim = n_pairs - p0 < window ? n_pairs - p0 : window;
    __syncthreads();
    for (int i = threadIdx.x; i < lim; i += 32 * DW_ROWS) {
      const int pr = p0 + i;
      const int ts = n_steps - 1 - pr / B, b = pr % B;      // ts = t - t0 - 1; pairs run t descending, b ascending
      const size_t rowi = (size_t)ts * B + b;
      s_words[i] = a.mask_row0[rowi * a.Wm + wc];
      s_off[i] = (uint32_t)ts * stride16 + (uint32_t)b * n16;
      if (GRADED) s_rowi[i] = (uint32_t)rowi;
    }
    __syncthreads();
    // this warp's row: the window's pairs in which it fired, in pair order
    int n_ev = 0;
    for (int sb = 0; sb < lim; sb += 32) {
      const uint32_t wd = sb + lane < lim ? s_words[sb + lane] : 0u;
      const bool on = (wd >> bit) & 1u;
      const uint32_t m = __ballot_sync(0xffffffffu, on);
      if (on) {
        const int slot = n_ev + __popc(m & ((1u << lane) - 1u));
        s_evw[slot] = s_off[sb + lane];
        if (GRADED) {   // the event's value: list start + events before its word + events before it in the word
          const size_t rowi = s_rowi[sb + lane];
          const uint32_t pos = a.off_row0[rowi] + a.pref_row0[rowi * a.Wm + wc] + __popc(wd & ((1u << bit) - 1u));
          s_valw[slot] = pos < a.cap ? a.vals[(rowi % B) * a.cap + pos] : 0.f;
        }
      }
      n_ev += __popc(m);
    }
    __syncwarp();
    if (row_ok) {
      // the listed delta rows stream through a per-warp ring of DW_STAGES groups of DW_GROUP rows
      const int n_groups = (n_ev + DW_GROUP - 1) / DW_GROUP;
      auto issue = [&](int g) {
        if (g < n_groups) {
#pragma unroll
          for (int q = 0; q < DW_GROUP; ++q) {
            const int e = g * DW_GROUP + q;
            if (e < n_ev) {
              const float4* d = delta_c + s_evw[e];
#pragma unroll
              for (int u = 0; u < U; ++u)
                if (colb + u * 128 < a.N) cp_async16(ring + (((g % DW_STAGES) * DW_GROUP + q) * U + u) * 32, d + u * 32);
            }
          }
        }
        cp_async_commit();
      };
      for (int g = 0; g < DW_STAGES - 1; ++g) issue(g);
      for (int g = 0; g < n_groups; ++g) {
        issue(g + DW_STAGES - 1);
        cp_async_wait<DW_STAGES - 1>();
#pragma unroll
        for (int q = 0; q < DW_GROUP; ++q) {
          if (g * DW_GROUP + q < n_ev) {
#pragma unroll
            for (int u = 0; u < U; ++u)
              if (colb + u * 128 < a.N) {
                const float4 dv = ring[(((g % DW_STAGES) * DW_GROUP + q) * U + u) * 32];
                if (GRADED) {
                  const float sv = s_valw[g * DW_GROUP + q];
                  acc[u].x = fmaf(sv, dv.x, acc[u].x); acc[u].y = fmaf(sv, dv.y, acc[u].y);
                  acc[u].z = fmaf(sv, dv.z, acc[u].z); acc[u].w = fmaf(sv, dv.w, acc[u].w);
                } else {
                  acc[u].x += dv.x; acc[u].y += dv.y; acc[u].z += dv.z; acc[u].w += dv.w;
                }
              }
          }
        }
      }
      cp_async_wait<0>();
    }
  }
  if (row_ok) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int c = colb + u * 128;
      if (c < a.N) *reinterpret_cast<float4*>(a.dW + (size_t)row * a.N + c) = acc[u];
    }
  }
}

// ------------------------------------------------------------------------------------------
// The same weight gradient with the deltas as the stationary operand (large layers).
//
// dw_kernel fetches a delta row from L2 once per event: on a network whose layers are thousands wide that is
// several times the bytes of dW itself and the L2 gather sets the time.  Here a CTA owns a slab of DWS_COLS
// columns and a group of DWS_ROWS presynaptic rows.  Per window of DWS_PAIRS (t, b) pairs it copies the slab
// delta[pair][columns] into shared memory once (128 KB) together with the spike words of its rows, and then every
// warp walks through rows of the group: the row's firing pattern over the window's pairs comes from four ballots
// over the spike words, the row's values of dW are read (the next rows of the warp already on their way), the slab
// rows of the pairs in which it fired are added in pair order (two 16-byte shared-memory reads and four packed
// additions per lane and event), and the row is written back.  Rows that did not fire in the window are not written.
// Per element the additions are those of dw_kernel in the same order (t descending, b ascending, starting from
// the stored value; a store and a reload between two windows do not change an fp32 value): the same bits.
// One CTA of 32 warps per SM: the event loop is bound by instruction issue, and a lane that owns eight columns
// halves the instructions per byte of a lane that owns four (measured on the largest benchmark network, per train
// step: 101 ms gathering, 91 ms with 128-column slabs, 58 ms with 256-column slabs and 32 warps).
constexpr int DWS_V = 2;          // 16-byte pieces of a row per lane
constexpr int DWS_COLS = 128 * DWS_V;   // columns per CTA
constexpr int DWS_PAIRS = 128;    // (t, b) pairs per window
constexpr int DWS_ROWS = 1024;    // presynaptic rows per CTA at most (DwParams::slab_rows: 1024, 512 or 256)
constexpr int DWS_WARPS = 32;
constexpr int DWS_BATCH = 2;      // rows of a warp whose dW values are in flight together (twice that with the prefetch)
// shared memory: the slab, the spike words of the row group, and for the graded cell the number of events before each
// of those words in its (step, sample) list
template <bool GRADED> constexpr size_t dws_smem_bytes() {
  return (size_t)DWS_PAIRS * DWS_COLS * sizeof(float) + (size_t)(DWS_ROWS / 32) * DWS_PAIRS * (sizeof(uint32_t) + (GRADED ? sizeof(uint16_t) : 0));
}

// Graded cell: an event multiplies the delta row by the event's value.  The value of (pair, row) sits in the value pool
// at the start of the pair's list + the events before the row's spike word + the events before the row inside the word;
// lane q looks up the value of pair 32 w + q while the ballots are taken, and the event loop hands it round by shuffle.
template <bool GRADED>
__global__ void __launch_bounds__(32 * DWS_WARPS) dw_slab_kernel(const __grid_constant__ DwParams p) {
  pdl_launch_dependents();
  const DwArgs& a = p.m[blockIdx.z];
  const int col0 = blockIdx.x * DWS_COLS, row0 = blockIdx.y * p.slab_rows;
  if (row0 >= a.N_pre || col0 >= a.N) return;
  pdl_wait();
  extern __shared__ float4 s_slab[];   // [DWS_PAIRS][DWS_V][32] float4, then the spike words [DWS_ROWS / 32][DWS_PAIRS]
  uint32_t* const s_words = reinterpret_cast<uint32_t*>(s_slab + (size_t)DWS_PAIRS * DWS_V * 32);
  uint16_t* const s_pref = reinterpret_cast<uint16_t*>(s_words + (size_t)(DWS_ROWS / 32) * DWS_PAIRS);   // graded only
  __shared__ uint32_t s_pair_row[DWS_PAIRS];   // (step, sample) row index ts * B + b of the window's pairs
  __shared__ uint32_t s_pair_off[GRADED ? DWS_PAIRS : 1];   // graded: start of the pair's list in its sample's pool
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int B = p.B, n_steps = p.n_steps, n_pairs = n_steps * B;
  const int wc0 = row0 >> 5;
  const int col = col0 + lane * 4;           // this lane's columns: col + 128 v .. + 3, v < DWS_V
  const int rows_here = a.N_pre - row0 < p.slab_rows ? a.N_pre - row0 : p.slab_rows;
  const uint32_t slab_lane = smem_u32(s_slab) + (uint32_t)lane * 16u;
  for (int p0 = 0; p0 < n_pairs; p0 += DWS_PAIRS) {
    const int lim = n_pairs - p0 < DWS_PAIRS ? n_pairs - p0 : DWS_PAIRS;
    __syncthreads();   // the previous window's readers are done
    if (tid < DWS_PAIRS) {
      const int pair = p0 + (tid < lim ? tid : 0);
      const int ts = n_steps - 1 - pair / B, b = pair % B;      // ts = t - t0 - 1; pairs run t descending, b ascending
      s_pair_row[tid] = (uint32_t)(ts * B + b);
      if (GRADED) s_pair_off[tid] = a.off_row0[ts * B + b];
    }
    __syncthreads();
    for (int pr = warp; pr < DWS_PAIRS; pr += DWS_WARPS) {   // a warp copies whole slab rows
      const uint32_t rowi = s_pair_row[pr];
      const float* const src = a.delta0 + (size_t)(rowi / B) * p.slot_stride + (size_t)(rowi % B) * a.N + col;
#pragma unroll
      for (int v = 0; v < DWS_V; ++v) {
        const bool real = pr < lim && col + 128 * v < a.N;
        cp_async16_or_zero(s_slab + (pr * DWS_V + v) * 32 + lane, real ? src + 128 * v : a.delta0, real);
      }
    }
    cp_async_commit();
    for (int i = tid; i < (p.slab_rows / 32) * DWS_PAIRS; i += 32 * DWS_WARPS) {
      const int jw = i / DWS_PAIRS, pr = i % DWS_PAIRS;
      uint32_t wd = 0u;
      uint16_t pf = 0;
      if (pr < lim && wc0 + jw < a.Wm) {
        wd = a.mask_row0[(size_t)s_pair_row[pr] * a.Wm + wc0 + jw];
        if (GRADED) pf = a.pref_row0[(size_t)s_pair_row[pr] * a.Wm + wc0 + jw];
      }
      s_words[i] = wd;
      if (GRADED) s_pref[i] = pf;
    }
    cp_async_wait<0>();
    __syncthreads();
    // warp w takes rows w, w + DWS_WARPS, ... of the group, DWS_BATCH of them at a time; the dW values of the next
    // batch are on their way while the current one is added to (rows that turn out not to have fired are read for
    // nothing, never written)
    float4 nxt[DWS_BATCH][DWS_V];
    auto fetch = [&](int r0) {
#pragma unroll
      for (int u = 0; u < DWS_BATCH; ++u) {
        const int r = r0 + u * DWS_WARPS;
#pragma unroll
        for (int v = 0; v < DWS_V; ++v) {
          nxt[u][v] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (r < rows_here && col + 128 * v < a.N)
            nxt[u][v] = *reinterpret_cast<const float4*>(a.dW + (size_t)(row0 + r) * a.N + col + 128 * v);
        }
      }
    };
    fetch(warp);
    for (int r0 = warp; r0 < rows_here; r0 += DWS_WARPS * DWS_BATCH) {
      unsigned long long acc[DWS_BATCH][DWS_V][2];   // two fp32 values per register pair
#pragma unroll
      for (int u = 0; u < DWS_BATCH; ++u)
#pragma unroll
        for (int v = 0; v < DWS_V; ++v) {
          acc[u][v][0] = (unsigned long long)__float_as_uint(nxt[u][v].x) | ((unsigned long long)__float_as_uint(nxt[u][v].y) << 32);
          acc[u][v][1] = (unsigned long long)__float_as_uint(nxt[u][v].z) | ((unsigned long long)__float_as_uint(nxt[u][v].w) << 32);
        }
      fetch(r0 + DWS_WARPS * DWS_BATCH);
#pragma unroll
      for (int u = 0; u < DWS_BATCH; ++u) {
        const int r = r0 + u * DWS_WARPS;
        const int jw = (r & (DWS_ROWS - 1)) >> 5;
        const uint32_t* const wds = s_words + (size_t)jw * DWS_PAIRS;
        bool any = false;
        uint32_t bits_w[DWS_PAIRS / 32];
        float val_w[DWS_PAIRS / 32];
#pragma unroll
        for (int w = 0; w < DWS_PAIRS / 32; ++w) {
          const uint32_t wd = wds[w * 32 + lane];
          const bool on = (wd >> (r & 31)) & 1u;
          bits_w[w] = __ballot_sync(0xffffffffu, on);
          any |= bits_w[w] != 0u;
          val_w[w] = 0.f;
          if (GRADED && on) {   // the value of this lane's pair for row r
            const int pr = w * 32 + lane;
            const uint32_t pos = s_pair_off[pr] + s_pref[jw * DWS_PAIRS + pr] + __popc(wd & ((1u << (r & 31)) - 1u));
            if (pos < a.cap) val_w[w] = a.vals[(size_t)(s_pair_row[pr] % B) * a.cap + pos];
          }
        }
#pragma unroll
        for (int w = 0; w < DWS_PAIRS / 32; ++w) {
          uint32_t bits = bits_w[w];
          const uint32_t base = slab_lane + (uint32_t)w * 32u * (DWS_COLS * 4u);
          while (bits) {   // one event: this lane's pieces of the pair's slab row, two packed operations each
            const uint32_t q = (uint32_t)__ffs(bits) - 1u;
            bits &= bits - 1u;
            unsigned long long vv = 0ull;
            if (GRADED) {
              const uint32_t sv = __float_as_uint(__shfl_sync(0xffffffffu, val_w[w], (int)q));
              vv = (unsigned long long)sv | ((unsigned long long)sv << 32);
            }
#pragma unroll
            for (int v = 0; v < DWS_V; ++v) {
              unsigned long long d01, d23;
              lds_2x64(base + q * (DWS_COLS * 4u) + v * 512u, d01, d23);
              if (GRADED) { fma_f32x2(acc[u][v][0], d01, vv); fma_f32x2(acc[u][v][1], d23, vv); }
              else { add_f32x2(acc[u][v][0], d01); add_f32x2(acc[u][v][1], d23); }
            }
          }
        }
        if (any && r < rows_here) {
#pragma unroll
          for (int v = 0; v < DWS_V; ++v)
            if (col + 128 * v < a.N)
              *reinterpret_cast<float4*>(a.dW + (size_t)(row0 + r) * a.N + col + 128 * v) =
                  make_float4(__uint_as_float((uint32_t)acc[u][v][0]), __uint_as_float((uint32_t)(acc[u][v][0] >> 32)),
                              __uint_as_float((uint32_t)acc[u][v][1]), __uint_as_float((uint32_t)(acc[u][v][1] >> 32)));
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Readout: logits = scale * c W_out, mean soft-max cross-entropy, and the gradients that
// leave it.  One small dense product per training step; plain fp32.
__global__ void __launch_bounds__(256)
readout_logits_kernel(const uint32_t* __restrict__ counts, int counts_are_float, const float* __restrict__ W_out,
                      int N_L, int N_out, float scale, float* __restrict__ logits) {
  extern __shared__ float s_part[];  // [8][N_out]
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int k = lane; k < N_out; k += 32) s_part[warp * N_out + k] = 0.f;
  __syncwarp();
  for (int i = warp; i < N_L; i += 8) {
    const uint32_t c = counts[(size_t)b * N_L + i];
    if (!c) continue;
    const float cf = counts_are_float ? __uint_as_float(c) : (float)c;
    for (int k = lane; k < N_out; k += 32) s_part[warp * N_out + k] = fmaf(cf, W_out[(size_t)i * N_out + k], s_part[warp * N_out + k]);
  }
  __syncthreads();
  for (int k = threadIdx.x; k < N_out; k += 256) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += s_part[w * N_out + k];
    logits[(size_t)b * N_out + k] = scale * s;
  }
}

__global__ void __launch_bounds__(256)
softmax_loss_kernel(const float* __restrict__ logits, const int32_t* __restrict__ targets, int B, int N_out,
                    float* __restrict__ dlogits, float* __restrict__ loss_out, uint32_t* __restrict__ status) {
  extern __shared__ float s_loss[];  // [B]
  for (int b = threadIdx.x; b < B; b += 256) {
    const float* z = logits + (size_t)b * N_out;
    float m = -INFINITY;
    for (int k = 0; k < N_out; ++k) m = fmaxf(m, z[k]);
    float se = 0.f;
    for (int k = 0; k < N_out; ++k) se += expf(z[k] - m);
    const float lse = m + logf(se);
    int tg = targets[b];
    if (tg < 0 || tg >= N_out) {   // never used as an index: the step reports it and its results are void
      atomicOr(status, STATUS_BAD_TARGET);
      tg = 0;
    }
    s_loss[b] = lse - z[tg];
    for (int k = 0; k < N_out; ++k)
      dlogits[(size_t)b * N_out + k] = (expf(z[k] - lse) - (k == tg ? 1.f : 0.f)) / (float)B;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int b = 0; b < B; ++b) s += s_loss[b];
    *loss_out = s / (float)B;
  }
}

// g_out[b, i] = scale * sum_k W_out[i, k] dlogits[b, k]
__global__ void __launch_bounds__(256)
readout_gout_kernel(const float* __restrict__ W_out, const float* __restrict__ dlogits, int B, int N_L, int N_out,
                    float scale, float* __restrict__ g_out) {
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= (size_t)B * N_L) return;
  const int b = (int)(idx / N_L), i = (int)(idx % N_L);
  float s = 0.f;
  for (int k = 0; k < N_out; ++k) s = fmaf(W_out[(size_t)i * N_out + k], dlogits[(size_t)b * N_out + k], s);
  g_out[idx] = scale * s;
}

// dW_out[i, k] = scale * sum_b c[b, i] dlogits[b, k]
__global__ void __launch_bounds__(256)
readout_dwout_kernel(const uint32_t* __restrict__ counts, int counts_are_float, const float* __restrict__ dlogits,
                     int B, int N_L, int N_out, float scale, float* __restrict__ dW_out) {
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= (size_t)N_L * N_out) return;
  const int i = (int)(idx / N_out), k = (int)(idx % N_out);
  float s = 0.f;
  for (int b = 0; b < B; ++b) {
    const uint32_t c = counts[(size_t)b * N_L + i];
    s = fmaf(counts_are_float ? __uint_as_float(c) : (float)c, dlogits[(size_t)b * N_out + k], s);
  }
  dW_out[idx] = scale * s;
}

}  // namespace snnk
