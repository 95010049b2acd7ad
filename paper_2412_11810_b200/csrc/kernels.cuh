// Device code of the BPTT step: spike compaction, event-driven forward step, surrogate-gradient
// backward step, sparse outer-product weight gradients, readout.  sm_100a, fp32.
//
// Arithmetic that decides spikes is written with explicit round-to-nearest intrinsics
// (__fadd_rn, __fmaf_rn, __fsub_rn, __fmul_rn) so that it is the same sequence of IEEE
// operations whatever the compiler flags: one accumulator per neuron, feed-forward events
// first, then recurrent events, each list in ascending presynaptic index, one fused
// multiply-add for the leak, one subtraction for the reset.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace snnk {

constexpr int MAXL = 8;
constexpr int FWD_THREADS = 128;            // each thread owns 4 adjacent neurons of one sample
constexpr int FWD_COLS = FWD_THREADS * 4;   // neurons per CTA
constexpr int LIST_CHUNK = 1024;            // events staged in shared memory at a time
constexpr int MAX_WORDS = 2048;             // 65536 neurons / 32
constexpr uint32_t STATUS_EVENT_OVERFLOW = 1u;

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

// ------------------------------------------------------------------------------------------
// Spike compaction ("Spike Generation" in its sparse representation): spike words -> ascending
// index list.  Step 1: exclusive prefix sum of the per-word popcounts over the whole row.
// Returns the number of set bits; s_pref[w] = number of set bits in words [0, w).
template <int NT>
__device__ uint32_t prefix_popcounts(const uint32_t* __restrict__ words, int n_words, uint32_t* s_pref,
                                     uint32_t* s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wpt = (n_words + NT - 1) / NT;
  const int w0 = tid * wpt;
  uint32_t sum = 0;
  for (int i = 0; i < wpt; ++i)
    if (w0 + i < n_words) sum += __popc(words[w0 + i]);
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
    if (w0 + i < n_words) { s_pref[w0 + i] = ex; ex += __popc(words[w0 + i]); }
  __syncthreads();
  return total;
}

// Step 2a: the part [c0, c0 + LIST_CHUNK) of the list into shared memory.
template <int NT>
__device__ void fill_chunk_from_words(const uint32_t* __restrict__ words, int n_words, const uint32_t* s_pref,
                                      uint32_t c0, uint32_t* s_list) {
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = words[w];
    if (!bits) continue;
    uint32_t p = s_pref[w];
    if (p >= c0 + LIST_CHUNK || p + __popc(bits) <= c0) continue;
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p >= c0 && p < c0 + LIST_CHUNK) s_list[p - c0] = (uint32_t)(w * 32 + bit);
      ++p;
    }
  }
}

// Step 2b: the whole list to global memory (entries past the capacity are dropped).
template <int NT>
__device__ void write_list_from_words(const uint32_t* __restrict__ words, int n_words, const uint32_t* s_pref,
                                      uint32_t* __restrict__ dst, uint32_t room) {
  for (int w = threadIdx.x; w < n_words; w += NT) {
    uint32_t bits = words[w];
    uint32_t p = s_pref[w];
    while (bits) {
      const int bit = __ffs(bits) - 1;
      bits &= bits - 1;
      if (p < room) dst[p] = (uint32_t)(w * 32 + bit);
      ++p;
    }
  }
}

// Stand-alone compaction of many rows: one CTA per row.
__global__ void __launch_bounds__(FWD_THREADS)
compact_rows_kernel(const uint32_t* __restrict__ masks, int n_words, uint32_t* __restrict__ idx_out,
                    int capacity, uint32_t* __restrict__ count_out) {
  __shared__ uint32_t s_pref[MAX_WORDS];
  __shared__ uint32_t s_warp[FWD_THREADS / 32];
  const size_t row = blockIdx.x;
  const uint32_t* words = masks + row * (size_t)n_words;
  const uint32_t total = prefix_popcounts<FWD_THREADS>(words, n_words, s_pref, s_warp);
  write_list_from_words<FWD_THREADS>(words, n_words, s_pref, idx_out + row * (size_t)capacity, (uint32_t)capacity);
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
  uint32_t* counts;           // [B][N] spike counts (last layer, generating mode) or null
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

// Adds the rows of W named by one event list to the accumulator, in list order.
// GEN: the list is compacted here from spike words; else it is read back from the pool.
template <bool GEN>
__device__ __forceinline__ void accumulate_list(const uint32_t* __restrict__ words, int n_words,
                                                uint32_t* __restrict__ pool, uint32_t* __restrict__ off,
                                                uint32_t cap, bool write_list, int B, int b,
                                                const float* __restrict__ W, int N, int col, bool active,
                                                float4& acc, uint32_t* s_list, uint32_t* s_pref,
                                                uint32_t* s_warp, uint32_t* status) {
  uint32_t total, start = 0;
  uint32_t* my_pool = pool + (size_t)b * cap;
  if (GEN) {
    total = prefix_popcounts<FWD_THREADS>(words, n_words, s_pref, s_warp);
    if (write_list) {
      start = off[b];
      const uint32_t room = cap - start;  // start <= cap always (clamped below)
      write_list_from_words<FWD_THREADS>(words, n_words, s_pref, my_pool + start, room);
      if (threadIdx.x == 0) {
        off[B + b] = start + (total < room ? total : room);
        if (total > room) atomicOr(status, STATUS_EVENT_OVERFLOW);
      }
    }
  } else {
    start = off[b];
    total = off[B + b] - start;
  }
  if (W == nullptr) return;
  const float* Wc = W + col;
  for (uint32_t c0 = 0; c0 < total; c0 += LIST_CHUNK) {
    const int n = (int)(total - c0 < (uint32_t)LIST_CHUNK ? total - c0 : (uint32_t)LIST_CHUNK);
    if (GEN) {
      fill_chunk_from_words<FWD_THREADS>(words, n_words, s_pref, c0, s_list);
    } else {
      for (int i = threadIdx.x; i < n; i += FWD_THREADS) s_list[i] = my_pool[start + c0 + i];
    }
    __syncthreads();
    if (active) {
      int e = 0;
      for (; e + 8 <= n; e += 8) {
        float4 w[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) w[u] = ldg4(Wc + (size_t)s_list[e + u] * N);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          acc.x = __fadd_rn(acc.x, w[u].x); acc.y = __fadd_rn(acc.y, w[u].y);
          acc.z = __fadd_rn(acc.z, w[u].z); acc.w = __fadd_rn(acc.w, w[u].w);
        }
      }
      for (; e < n; ++e) {
        const float4 w = ldg4(Wc + (size_t)s_list[e] * N);
        acc.x = __fadd_rn(acc.x, w.x); acc.y = __fadd_rn(acc.y, w.y);
        acc.z = __fadd_rn(acc.z, w.z); acc.w = __fadd_rn(acc.w, w.w);
      }
    }
    __syncthreads();
  }
}

template <bool GEN>
__global__ void __launch_bounds__(FWD_THREADS) fwd_step_kernel(const __grid_constant__ FwdParams p) {
  const FwdLayer& L = p.lay[blockIdx.z];
  if (L.mode == 0) return;
  const int col0 = blockIdx.x * FWD_COLS;
  if (col0 >= L.N) return;
  const int b = blockIdx.y, B = p.B;
  const bool tile0 = blockIdx.x == 0;
  __shared__ uint32_t s_list[LIST_CHUNK];
  __shared__ uint32_t s_pref[MAX_WORDS];
  __shared__ uint32_t s_warp[FWD_THREADS / 32];
  const int col = col0 + threadIdx.x * 4;
  const bool active = col < L.N;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);

  if (L.mode == 2) {  // after the last step: only store the list of the final spikes
    if (GEN && tile0)
      accumulate_list<true>(L.rec_mask + (size_t)b * L.W, L.W, L.rec_pool, L.rec_off, L.rec_cap, true, B, b,
                            nullptr, L.N, col, false, acc, s_list, s_pref, s_warp, p.status);
    return;
  }
  // feed-forward events: layer below, same step
  accumulate_list<GEN>(GEN ? L.ff_mask + (size_t)b * L.W_pre : nullptr, L.W_pre, L.ff_pool, L.ff_off, L.ff_cap,
                       tile0 && L.write_ff_list, B, b, L.W_ff, L.N, col, active, acc, s_list, s_pref, s_warp,
                       p.status);
  // recurrent events: own layer, previous step
  accumulate_list<GEN>(GEN ? L.rec_mask + (size_t)b * L.W : nullptr, L.W, L.rec_pool, L.rec_off, L.rec_cap, tile0,
                       B, b, L.W_rec, L.N, col, active, acc, s_list, s_pref, s_warp, p.status);

  // leak, reset by subtraction of the previous step's own spike, threshold
  uint32_t nib = 0;
  if (active) {
    const size_t k = (size_t)b * L.N + col;
    const float4 vp = *reinterpret_cast<const float4*>(L.V_prev + k);
    const uint32_t pw = L.rec_mask[(size_t)b * L.W + (col >> 5)] >> (col & 31);
    float4 v;
    v.x = __fsub_rn(__fmaf_rn(p.alpha, vp.x, acc.x), __fmul_rn(p.theta, (float)(pw & 1u)));
    v.y = __fsub_rn(__fmaf_rn(p.alpha, vp.y, acc.y), __fmul_rn(p.theta, (float)((pw >> 1) & 1u)));
    v.z = __fsub_rn(__fmaf_rn(p.alpha, vp.z, acc.z), __fmul_rn(p.theta, (float)((pw >> 2) & 1u)));
    v.w = __fsub_rn(__fmaf_rn(p.alpha, vp.w, acc.w), __fmul_rn(p.theta, (float)((pw >> 3) & 1u)));
    *reinterpret_cast<float4*>(L.V_out + k) = v;
    if (L.V_keep) *reinterpret_cast<float4*>(L.V_keep + k) = v;
    if (L.V_dbg) *reinterpret_cast<float4*>(L.V_dbg + k) = v;
    if (GEN) {
      nib = (v.x > p.theta ? 1u : 0u) | (v.y > p.theta ? 2u : 0u) | (v.z > p.theta ? 4u : 0u) |
            (v.w > p.theta ? 8u : 0u);
      if (L.counts && nib) {
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

// ------------------------------------------------------------------------------------------
// Backward step: delta^l_t = g_S sigma'(V^l_t - theta) + alpha delta^l_{t+1}, with
// g_S = g_out + W_ff^{l+1} delta^{l+1}_t + W_rec^l delta^l_{t+1} - theta delta^l_{t+1}.
// A warp owns R rows i of the weight matrices and all lanes split the contraction index;
// R * BT partial sums per lane are reduced across the warp in a fixed tree.
struct BwdLayer {
  const float* W_rec;     // [N][N]
  const float* W_ffa;     // W_ff of the layer above [N][N_post] or null
  float* V_delta;         // [B][N]: V_t on entry, delta_t on exit
  const float* d_next;    // [B][N]      delta^l_{t+1}
  const float* d_above;   // [B][N_post] delta^{l+1}_t or null
  const float* g_out;     // [B][N] or null
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

constexpr int BWD_WARPS = 4;

__device__ __forceinline__ float surrogate_grad(float v, float theta, float beta, int surrogate, int cell) {
  const float x = v - theta;
  if (cell == 1) return x > 0.f ? 1.f : 0.f;
  if (surrogate == 0) {
    const float d = fmaf(beta, fabsf(x), 1.f);
    return 1.f / (d * d);
  }
  const float s = 1.f / (1.f + expf(-beta * x));
  return beta * s * (1.f - s);
}

// Sum over the warp of 32 per-lane values; on return lane i holds the total of value i.
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[32], int lane) {
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const bool upper = (lane & s) != 0;
#pragma unroll
    for (int j = 0; j < s; ++j) {
      const float send = upper ? v[j] : v[j + s];
      const float keep = upper ? v[j + s] : v[j];
      v[j] = keep + __shfl_xor_sync(0xffffffffu, send, s);
    }
  }
  return v[0];
}

template <int BT, int R>
__device__ __forceinline__ void dot_rows(const float* __restrict__ W, int ld, int row0, int n_rows,
                                         const float* __restrict__ d, int b0, int B, int K, int lane,
                                         float (&acc)[32]) {
  static_assert(BT * R == 32, "one value per lane after the reduction");
  if (W == nullptr) return;
  for (int k = lane * 4; k < K; k += 128) {
    float4 w[R];
#pragma unroll
    for (int r = 0; r < R; ++r)
      w[r] = row0 + r < n_rows ? ldg4(W + (size_t)(row0 + r) * ld + k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int bb = 0; bb < BT; ++bb) {
      const float4 dv = b0 + bb < B ? ldg4(d + (size_t)(b0 + bb) * K + k) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float a = acc[r * BT + bb];
        a = fmaf(w[r].x, dv.x, a); a = fmaf(w[r].y, dv.y, a);
        a = fmaf(w[r].z, dv.z, a); a = fmaf(w[r].w, dv.w, a);
        acc[r * BT + bb] = a;
      }
    }
  }
}

template <int BT, int R>
__global__ void __launch_bounds__(BWD_WARPS * 32) bwd_step_kernel(const __grid_constant__ BwdParams p) {
  const BwdLayer& L = p.lay[blockIdx.z];
  if (L.mode == 0) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row0 = (blockIdx.x * BWD_WARPS + warp) * R;
  if (row0 >= L.N) return;
  for (int b0 = 0; b0 < p.B; b0 += BT) {
    float acc[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) acc[i] = 0.f;
    dot_rows<BT, R>(L.W_ffa, L.N_post, row0, L.N, L.d_above, b0, p.B, L.N_post, lane, acc);
    dot_rows<BT, R>(L.W_rec, L.N, row0, L.N, L.d_next, b0, p.B, L.N, lane, acc);
    const float sum = warp_transpose_reduce(acc, lane);
    const int i = row0 + lane / BT, b = b0 + lane % BT;
    if (i < L.N && b < p.B) {
      const size_t k = (size_t)b * L.N + i;
      const float dn = L.d_next[k];
      float g = sum + (L.g_out ? L.g_out[k] : 0.f);
      if (p.cell == 0) g = fmaf(-p.theta, dn, g);
      const float sp = surrogate_grad(L.V_delta[k], p.theta, p.beta, p.surrogate, p.cell);
      const float dl = fmaf(g, sp, p.alpha * dn);
      L.V_delta[k] = dl;
      if (L.carry_out) L.carry_out[k] = dl;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Sparse outer-product weight gradient over a run of steps t = t1 .. t0+1:
//   dW[j, :] += delta_t[b, :]   for every (t, b) in which presynaptic neuron j was active,
// accumulated per element in the fixed order t descending, b ascending, starting from the
// value already in dW.  A CTA owns 32 presynaptic rows (one spike word) and a column tile.
struct DwArgs {
  float* dW;                 // [N_pre][N]
  const uint32_t* mask_row0; // spike words of the presynaptic layer for t = t0+1: [(t-t0-1)][B][Wm]
  const float* delta0;       // delta of step t0+1: delta(t, b) = delta0 + (t-t0-1) * slot_stride + b * N
  size_t slot_stride;        // floats between consecutive steps
  int N_pre, N, Wm, B, n_steps;
};

template <int U>
__global__ void __launch_bounds__(256) dw_kernel(const DwArgs a) {
  __shared__ uint32_t s_words[256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wc = blockIdx.y;                 // spike word column = 32 presynaptic rows
  const int rowb = wc * 32 + warp * 4;       // this warp's 4 rows
  const int colb = blockIdx.x * (128 * U) + lane * 4;
  float4 acc[4][U];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int c = colb + u * 128;
      acc[r][u] = (rowb + r < a.N_pre && c < a.N)
                      ? *reinterpret_cast<const float4*>(a.dW + (size_t)(rowb + r) * a.N + c)
                      : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  const int n_pairs = a.n_steps * a.B;
  for (int p0 = 0; p0 < n_pairs; p0 += 256) {
    __syncthreads();
    {
      const int pr = p0 + threadIdx.x;
      uint32_t w = 0;
      if (pr < n_pairs) {
        const int ts = a.n_steps - 1 - pr / a.B, b = pr % a.B;   // ts = t - t0 - 1, t descending
        w = a.mask_row0[((size_t)ts * a.B + b) * a.Wm + wc];
      }
      s_words[threadIdx.x] = w;
    }
    __syncthreads();
    const int lim = n_pairs - p0 < 256 ? n_pairs - p0 : 256;
    for (int sb = 0; sb < lim; sb += 32) {
      const uint32_t wd = s_words[sb + lane] >> (warp * 4);
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        uint32_t m = __ballot_sync(0xffffffffu, (wd >> r) & 1u);
        while (m) {
          const int q = __ffs(m) - 1;
          m &= m - 1;
          const int pr = p0 + sb + q;
          const int ts = a.n_steps - 1 - pr / a.B, b = pr % a.B;
          const float* d = a.delta0 + (size_t)ts * a.slot_stride + (size_t)b * a.N + colb;
#pragma unroll
          for (int u = 0; u < U; ++u)
            if (colb + u * 128 < a.N) {
              const float4 dv = ldg4(d + u * 128);
              acc[r][u].x += dv.x; acc[r][u].y += dv.y; acc[r][u].z += dv.z; acc[r][u].w += dv.w;
            }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int c = colb + u * 128;
      if (rowb + r < a.N_pre && c < a.N)
        *reinterpret_cast<float4*>(a.dW + (size_t)(rowb + r) * a.N + c) = acc[r][u];
    }
}

// ------------------------------------------------------------------------------------------
// Readout: logits = scale * c W_out, mean soft-max cross-entropy, and the gradients that
// leave it.  One small dense product per training step; plain fp32.
__global__ void __launch_bounds__(256)
readout_logits_kernel(const uint32_t* __restrict__ counts, const float* __restrict__ W_out, int N_L, int N_out,
                      float scale, float* __restrict__ logits) {
  extern __shared__ float s_part[];  // [8][N_out]
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int k = lane; k < N_out; k += 32) s_part[warp * N_out + k] = 0.f;
  __syncwarp();
  for (int i = warp; i < N_L; i += 8) {
    const uint32_t c = counts[(size_t)b * N_L + i];
    if (!c) continue;
    const float cf = (float)c;
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
                    float* __restrict__ dlogits, float* __restrict__ loss_out) {
  extern __shared__ float s_loss[];  // [B]
  for (int b = threadIdx.x; b < B; b += 256) {
    const float* z = logits + (size_t)b * N_out;
    float m = -INFINITY;
    for (int k = 0; k < N_out; ++k) m = fmaxf(m, z[k]);
    float se = 0.f;
    for (int k = 0; k < N_out; ++k) se += expf(z[k] - m);
    const float lse = m + logf(se);
    const int tg = targets[b];
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
readout_dwout_kernel(const uint32_t* __restrict__ counts, const float* __restrict__ dlogits, int B, int N_L,
                     int N_out, float scale, float* __restrict__ dW_out) {
  const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (idx >= (size_t)N_L * N_out) return;
  const int i = (int)(idx / N_out), k = (int)(idx % N_out);
  float s = 0.f;
  for (int b = 0; b < B; ++b) s = fmaf((float)counts[(size_t)b * N_L + i], dlogits[(size_t)b * N_out + k], s);
  dW_out[idx] = scale * s;
}

}  // namespace snnk
