// C ABI and executor: validates arguments, carves the caller's workspaces, and runs the
// schedule of Fig. 1 (forward, recomputation passes, backward, checkpoint copies) as kernel
// launches on the main stream and copies on the side stream.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/snn.h"
#include "kernels.cuh"
#include "tc_gemm.cuh"

using namespace snnk;

struct snn_net {
  std::vector<int32_t> sizes;  // N_0, N_1..N_L, N_out
  int L = 0;
  float tau = 0, theta = 0, beta = 0, scale = 0, alpha = 0;
  int surrogate = 0, cell = 0;
  std::string err;
  size_t dev_peak = 0, pin_peak = 0;
  snn_memory_stats stats{};
  // layout of the last step, for inspection
  std::vector<snn_event_layout> ev_layout;
  cudaEvent_t ev_main = nullptr;
  cudaEvent_t ev_window[2] = {nullptr, nullptr};   // completion of the last copy of each event window (spilled events)
  std::vector<cudaEvent_t> copy_events;    // one per checkpoint copy in flight, grown on demand
  std::vector<cudaEvent_t> timing_events;  // grown on demand, reused by every timed step
  snn_phase_times phases{};
  int device = -1;                         // device the two figures below were asked of
  int coop_sms = -1;                       // SMs usable by a cooperative launch (-1: not asked yet)
  int fwd_segment_capacity[2] = {-1, -1};   // CTAs of fwd_segment_kernel the device holds at once with a deep / shallow copy ring (-1: not asked yet)
  int bwd_stream_capacity[6] = {-1, -1, -1, -1, -1, -1};   // the same for the six instances of bwd_stream_kernel
};

namespace {

// A named range on the profiler's timeline (NVTX; costs nothing while no tool is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

snn_status fail(snn_net* net, snn_status st, const char* fmt, ...) {
  if (net) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    net->err = buf;
  }
  return st;
}

constexpr size_t ALIGN = 256;
constexpr int BWD_RUN = 32;   // steps per run of the layer-by-layer backward pass
size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

struct Layout {
  size_t status, progress, logits, dlogits, g_out, counts, carry[2], vcarry, in_stage, tg_stage;
  size_t off[MAXL + 1], pool[MAXL + 1], mask[MAXL + 1];
  size_t vals[MAXL + 1], pref[MAXL + 1], act[MAXL + 1], in_words;   // graded cell only
  uint32_t cap[MAXL + 1];
  int words[MAXL + 1];
  size_t slots, state_bytes, layer_off[MAXL + 1];  // layer_off in floats within a state
  size_t event_bytes, total;
  bool spill;              // event windows per remote segment, the rest in pinned memory
  int ev_steps;            // steps per event window (the whole sequence without spilling)
  int ev_segments;         // windows the sequence consists of
  size_t ev_base, ev_window_bytes;
  size_t gff;            // [BWD_RUN * B][max N] product W_ff delta of the layer above for a run of steps (large nets),
                         // as up to TCG_MAX_KSPLIT partial products gff_stride floats apart
  size_t gff_stride;
  bool layer_major;      // backward goes layer by layer over runs of steps, with that product batched over time
  bool weights_resident; // all weight matrices together stay in L2
  size_t rows_ev;        // event words of a run of recomputed steps (refwd_rows_kernel), then the raw words
  size_t rows_ev_words;  // words of each of the two halves
  size_t rows_ev_stride; // words per block of 32 rows: the pairs of the longest run, rounded up
  size_t tier2;          // DOUBLE_LOCAL: the second checkpoint tier, in device memory
  int n_local, n_remote;
  bool tier2_on_device;
};

// Cluster size of the wavefront backward kernels along the contraction index: enough CTAs to fill the GPU (one wave:
// two 256-thread CTAs or one 512-thread CTA per SM on 148 SMs), at least one full warp pass (128 values) per rank; a
// function of the network sizes and the batch only.
int backward_cluster_size(const std::vector<int>& sz, int L, int B) {
  int maxN = 0;
  for (int l = 1; l <= L; ++l) maxN = std::max(maxN, sz[l]);
  int minN = maxN;
  for (int l = 1; l <= L; ++l) minN = std::min(minN, sz[l]);
  const int tiles = (maxN + BWD_TM - 1) / BWD_TM;
  const int wave = B <= 16 ? 296 : 148;
  int CS = 1;
  while (CS < 8 && tiles * L * CS * 2 <= wave && minN / (4 * CS * 2) >= 32) CS *= 2;
  return CS;
}
// Dynamic shared memory bwd_segment_kernel needs: the largest slice of W_ff(l+1) and W_rec a cluster rank keeps
// resident (32 rows x its share of the contraction index) and the staging region.
size_t backward_segment_smem(const std::vector<int>& sz, int L, int B, int CS) {
  const int nwarp = B <= 16 ? 8 : 16;
  size_t res_floats = 0;
  for (int l = 1; l <= L; ++l) {
    const int q_rec = sz[l] / 4, q_ff = (l < L ? sz[l + 1] : 0) / 4;
    for (int r = 0; r < CS; ++r) {
      const int k_rec = (int)((long long)q_rec * (r + 1) / CS) * 4 - (int)((long long)q_rec * r / CS) * 4;
      const int k_ff = (int)((long long)q_ff * (r + 1) / CS) * 4 - (int)((long long)q_ff * r / CS) * 4;
      res_floats = std::max(res_floats, (size_t)BWD_TM * bwd_resident_ld(k_ff, k_rec, nwarp));
    }
  }
  const size_t region = B <= 8 ? bwd_segment_region_floats<1, 8>() : B <= 16 ? bwd_segment_region_floats<2, 8>()
                                                                           : bwd_segment_region_floats<4, 16>();
  return 4 * (res_floats + region);
}
constexpr size_t BWD_SEGMENT_SMEM_MAX = (size_t)218 << 10;

bool compute_layout(const snn_net* net, int T, int B, const snn_ckpt* ck, float max_activity, uint32_t flags,
                    Layout& lo, std::string& why) {
  const int L = net->L;
  const auto& sz = net->sizes;
  int n_ops = 0;
  if (snn_plan(T, ck, nullptr, 0, &n_ops, &lo.n_local, &lo.n_remote) != SNN_OK) {
    why = "invalid checkpoint intervals";
    return false;
  }
  size_t cur = 0;
  auto take = [&](size_t bytes) { size_t o = cur; cur = align_up(cur + bytes); return o; };
  const int N_L = sz[L], N_out = sz[L + 1];
  size_t sumN = 0;
  for (int l = 1; l <= L; ++l) { lo.layer_off[l] = (size_t)B * sumN; sumN += sz[l]; }
  lo.state_bytes = 4 * (size_t)B * sumN;
  lo.status = take(256);
  lo.progress = take(4 * (size_t)MAXL * B);   // per (layer, sample): finished (tile, step) pairs of a forward launch
  lo.logits = take(4 * (size_t)B * N_out);
  lo.dlogits = take(4 * (size_t)B * N_out);
  lo.g_out = take(4 * (size_t)B * N_L);
  lo.counts = take(4 * (size_t)B * N_L);
  lo.carry[0] = take(lo.state_bytes);
  lo.carry[1] = take(lo.state_bytes);
  lo.vcarry = take(lo.state_bytes);   // last state of a re-forward run, start of the next
  lo.words[0] = (sz[0] + 31) / 32;
  const bool graded = net->cell == SNN_CELL_GRADED;
  // staging of input and targets that arrive in host memory: only then
  const bool host_input = (flags & SNN_FLAG_INPUT_ON_HOST) != 0;
  lo.in_stage = host_input ? take(4 * (size_t)T * B * (graded ? sz[0] : lo.words[0])) : 0;
  lo.in_words = graded ? take(4 * (size_t)T * B * lo.words[0]) : 0;
  lo.tg_stage = host_input ? take(4 * (size_t)B) : 0;
  // Events (index lists, their offsets, spike words; values for the graded cell).  Normally the events of the whole
  // sequence stay in device memory.  With SNN_FLAG_SPILL_EVENTS (REMOTE, DOUBLE) the device holds two windows of
  // one remote segment each (the one in use and the one being copied), and every segment's window goes to pinned
  // memory behind the forward pass and comes back ahead of its backward pass.  Within a window rows are indexed by
  // the step relative to the segment's first state and list offsets restart at zero.
  lo.spill = (flags & SNN_FLAG_SPILL_EVENTS) && (ck->strategy == SNN_REMOTE || ck->strategy == SNN_DOUBLE);
  lo.ev_steps = T;
  if (lo.spill) lo.ev_steps = std::min(T, ck->strategy == SNN_DOUBLE ? ck->remote_chunk_size : ck->chunk_size);
  lo.ev_segments = (T + lo.ev_steps - 1) / lo.ev_steps;
  const int Tw = lo.ev_steps;
  const size_t ev0 = cur;
  for (int l = 0; l <= L; ++l) {
    lo.words[l] = (sz[l] + 31) / 32;
    const double want = std::ceil((double)max_activity * sz[l] * Tw) + sz[l];
    if (want > 4.0e9) { why = "event pool per sample exceeds 32-bit offsets"; return false; }
    lo.cap[l] = (uint32_t)want;
    lo.off[l] = take(4 * (size_t)(Tw + 2) * B);
    lo.pool[l] = take(4 * (size_t)B * lo.cap[l]);
    lo.mask[l] = l == 0 ? 0 : take(4 * (size_t)(Tw + 1) * B * lo.words[l]);
    lo.vals[l] = graded ? take(4 * (size_t)B * lo.cap[l]) : 0;
    lo.pref[l] = graded ? take(2 * (size_t)(Tw + 2) * B * lo.words[l]) : 0;
  }
  lo.ev_base = ev0;
  lo.ev_window_bytes = cur - ev0;
  if (lo.spill) take(lo.ev_window_bytes);   // the second window
  lo.event_bytes = cur - ev0;
  for (int l = 0; l <= L; ++l) lo.act[l] = (graded && l > 0) ? take(4 * (size_t)2 * B * sz[l]) : 0;
  {
    // Networks whose weight slices do not fit the shared memory of the segment kernel: multiplying by W_ff once per
    // run of steps (one product on the tensor cores, W_ff streamed once) instead of once per step pays for giving
    // up the layer wavefront in the backward pass.  A function of the sizes and the batch only.
    size_t wbytes = 0;
    int maxN = 0;
    for (int l = 1; l <= L; ++l) { wbytes += 4 * ((size_t)sz[l - 1] * sz[l] + (size_t)sz[l] * sz[l]); maxN = std::max(maxN, sz[l]); }
    lo.weights_resident = wbytes <= ((size_t)96 << 20);
    lo.layer_major = L > 1 && (!lo.weights_resident ||
                               backward_segment_smem(sz, L, B, backward_cluster_size(sz, L, B)) > BWD_SEGMENT_SMEM_MAX);
    lo.gff_stride = (size_t)BWD_RUN * B * maxN;
    lo.gff = L > 1 ? take(4 * lo.gff_stride * TCG_MAX_KSPLIT) : 0;
  }
  lo.rows_ev = 0; lo.rows_ev_words = 0; lo.rows_ev_stride = 0;
  if (ck->strategy != SNN_STANDARD) {
    // one word per (32 presynaptic rows, pair) for the pairs of a run (at most chunk_size steps), twice
    const int Kc = std::min(std::max(ck->chunk_size, 1), T);
    const size_t stride = ((size_t)Kc * B + RR_MAX_PB - 1) / RR_MAX_PB * RR_MAX_PB;
    size_t blocks = 0;
    for (int l = 1; l <= L; ++l) blocks += (size_t)lo.words[l - 1] + lo.words[l];
    lo.rows_ev_stride = stride;
    lo.rows_ev_words = stride * blocks;
    lo.rows_ev = take((graded ? 11 : 2) * 4 * lo.rows_ev_words);   // graded cell: counts, two words of rows, eight values
  }
  lo.slots = take((size_t)lo.n_local * lo.state_bytes);
  lo.tier2_on_device = ck->strategy == SNN_DOUBLE_LOCAL;
  lo.tier2 = lo.tier2_on_device ? take((size_t)lo.n_remote * lo.state_bytes) : 0;
  lo.total = cur;
  return true;
}

constexpr size_t RESIDENT_SMEM_MAX = (size_t)200 << 10;   // most dynamic shared memory fwd_resident_kernel is given

#define CUDA_TRY(expr)                                                                         \
  do {                                                                                         \
    cudaError_t e_ = (expr);                                                                   \
    if (e_ != cudaSuccess)                                                                     \
      return fail(net, SNN_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_));          \
  } while (0)

}  // namespace

extern "C" snn_status snn_create(const snn_config* cfg, snn_net** out) {
  if (!cfg || !out || !cfg->sizes || cfg->n_sizes < 3) return SNN_ERR_INVALID_ARG;
  const int L = cfg->n_sizes - 2;
  if (L > SNN_MAX_LAYERS) return SNN_ERR_UNSUPPORTED;
  for (int i = 0; i < cfg->n_sizes; ++i)
    if (cfg->sizes[i] < 1) return SNN_ERR_INVALID_ARG;
  for (int l = 1; l <= L; ++l)
    if (cfg->sizes[l] % 4 != 0 || cfg->sizes[l] > SNN_MAX_NEURONS) return SNN_ERR_UNSUPPORTED;
  if (cfg->sizes[0] > SNN_MAX_NEURONS) return SNN_ERR_UNSUPPORTED;
  if (!(cfg->tau_mem > 0) || !(cfg->surrogate_beta > 0)) return SNN_ERR_INVALID_ARG;
  if (cfg->surrogate != SNN_SURR_FAST_SIGMOID && cfg->surrogate != SNN_SURR_SIGMOID &&
      cfg->surrogate != SNN_SURR_TRIANGLE)
    return SNN_ERR_INVALID_ARG;
  if (cfg->cell != SNN_CELL_LIF && cfg->cell != SNN_CELL_GRADED) return SNN_ERR_INVALID_ARG;
  snn_net* n = new snn_net();
  n->sizes.assign(cfg->sizes, cfg->sizes + cfg->n_sizes);
  n->L = L;
  n->tau = cfg->tau_mem; n->theta = cfg->threshold; n->beta = cfg->surrogate_beta;
  n->scale = cfg->readout_scale; n->surrogate = cfg->surrogate; n->cell = cfg->cell;
  n->alpha = (float)std::exp(-1.0 / (double)cfg->tau_mem);
  *out = n;
  return SNN_OK;
}

extern "C" void snn_destroy(snn_net* net) {
  if (!net) return;
  if (net->ev_main) cudaEventDestroy(net->ev_main);
  for (cudaEvent_t e : net->ev_window)
    if (e) cudaEventDestroy(e);
  for (auto& e : net->copy_events) cudaEventDestroy(e);
  for (auto& e : net->timing_events) cudaEventDestroy(e);
  delete net;
}

extern "C" float snn_alpha(const snn_net* net) { return net ? net->alpha : 0.f; }

extern "C" int32_t snn_debug_checks_enabled(void) {
#ifdef SNN_DEBUG_CHECKS
  return 1;
#else
  return 0;
#endif
}

extern "C" const char* snn_last_error(const snn_net* net) { return net ? net->err.c_str() : "null net"; }

extern "C" snn_status snn_workspace_query(const snn_net* net, int32_t T, int32_t B, const snn_ckpt* ckpt,
                                          float max_activity, size_t* device_bytes, size_t* pinned_bytes) {
  return snn_workspace_query_flags(net, T, B, ckpt, max_activity, 0u, device_bytes, pinned_bytes);
}

extern "C" snn_status snn_workspace_query_flags(const snn_net* net, int32_t T, int32_t B, const snn_ckpt* ckpt,
                                                float max_activity, uint32_t flags, size_t* device_bytes,
                                                size_t* pinned_bytes) {
  if (!net || !ckpt || T < 1 || B < 1 || !(max_activity > 0.f) || max_activity > 1.f) return SNN_ERR_INVALID_ARG;
  Layout lo;
  std::string why;
  if (!compute_layout(net, T, B, ckpt, max_activity, flags, lo, why))
    return fail(const_cast<snn_net*>(net), SNN_ERR_INVALID_ARG, "%s", why.c_str());
  if (device_bytes) *device_bytes = lo.total;
  if (pinned_bytes) *pinned_bytes = (lo.tier2_on_device ? 0 : (size_t)lo.n_remote * lo.state_bytes) +
                                    (lo.spill ? (size_t)lo.ev_segments * lo.ev_window_bytes : 0);
  return SNN_OK;
}

extern "C" snn_status snn_peak_memory(const snn_net* net, size_t* device_peak_bytes, size_t* pinned_peak_bytes) {
  if (!net) return SNN_ERR_INVALID_ARG;
  if (device_peak_bytes) *device_peak_bytes = net->dev_peak;
  if (pinned_peak_bytes) *pinned_peak_bytes = net->pin_peak;
  return SNN_OK;
}

extern "C" snn_status snn_memory_stats_get(const snn_net* net, snn_memory_stats* out) {
  if (!net || !out) return SNN_ERR_INVALID_ARG;
  *out = net->stats;
  return SNN_OK;
}

extern "C" snn_status snn_phase_times_get(const snn_net* net, snn_phase_times* out) {
  if (!net || !out) return SNN_ERR_INVALID_ARG;
  *out = net->phases;
  return SNN_OK;
}

extern "C" snn_status snn_get_event_layout(const snn_net* net, int32_t layer, snn_event_layout* out) {
  if (!net || !out || layer < 0 || layer >= (int)net->ev_layout.size()) return SNN_ERR_INVALID_ARG;
  *out = net->ev_layout[layer];
  return SNN_OK;
}

extern "C" snn_status snn_compact_spikes(const uint32_t* masks, int32_t n_rows, int32_t n_words, uint32_t* idx_out,
                                         int32_t capacity, uint32_t* count_out, void* stream) {
  if (n_rows < 0 || n_words < 0 || capacity < 0) return SNN_ERR_INVALID_ARG;
  if (n_words > MAX_WORDS) return SNN_ERR_UNSUPPORTED;
  if (n_rows == 0) return SNN_OK;
  if (!masks && n_words > 0) return SNN_ERR_INVALID_ARG;
  if (!count_out || (!idx_out && capacity > 0)) return SNN_ERR_INVALID_ARG;
  compact_rows_kernel<<<n_rows, FWD_THREADS, 0, (cudaStream_t)stream>>>(masks, n_words, idx_out, capacity, count_out);
  return cudaGetLastError() == cudaSuccess ? SNN_OK : SNN_ERR_CUDA;
}

namespace {

struct Exec {
  snn_net* net;
  const snn_step_args* a;
  Layout lo;
  char* ws;
  cudaStream_t main, side;
  int L, B, T;
  int launches = 0, d2h = 0, h2d = 0;
  int carry_cur = 0;
  std::vector<int> slot_event;   // per local slot: index of the copy event it waits on, or -1
  int copies_in_flight = 0;
  bool remote_tier;
  bool timed = false;
  struct Span { int phase, ev0, ev1, launches; };
  std::vector<Span> spans;
  int ev_used = 0;

  // Brackets [begin_span, end_span) on the main stream with two events of the net's pool.
  int begin_span(int phase, cudaStream_t st = nullptr) {
    if (!timed) return -1;
    if (!st) st = main;
    auto& pool_ev = net->timing_events;
    while ((int)pool_ev.size() < ev_used + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { timed = false; return -1; }
      pool_ev.push_back(e);
    }
    cudaEventRecord(pool_ev[ev_used], st);
    spans.push_back(Span{phase, ev_used, ev_used + 1, launches});
    ev_used += 2;
    return (int)spans.size() - 1;
  }
  void end_span(int id, cudaStream_t st = nullptr) {
    if (id < 0) return;
    cudaEventRecord(net->timing_events[spans[id].ev1], st ? st : main);
    spans[id].launches = st ? 1 : launches - spans[id].launches;
  }
  void collect_spans() {
    net->phases = snn_phase_times{};
    for (const Span& sp : spans) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, net->timing_events[sp.ev0], net->timing_events[sp.ev1]) == cudaSuccess)
        net->phases.ms[sp.phase] += ms;
      net->phases.launches[sp.phase] += sp.launches;
    }
  }

  template <class Tp> Tp* at(size_t off) const { return reinterpret_cast<Tp*>(ws + off); }
  mutable bool debug_violation = false;   // bounds-checked build: the plan named a state slot the layout does not have
  float* slot(int s, int l) const {
#ifdef SNN_DEBUG_CHECKS
    if (s < 0 || s >= lo.n_local) { debug_violation = true; s = 0; }
#endif
    return at<float>(lo.slots + (size_t)s * lo.state_bytes) + lo.layer_off[l];
  }
  float* carry(int which, int l) const { return at<float>(lo.carry[which]) + lo.layer_off[l]; }
  bool graded() const { return net->cell == SNN_CELL_GRADED; }
  const void* in_base() const { return (a->flags & SNN_FLAG_INPUT_ON_HOST) ? (const void*)(ws + lo.in_stage) : a->input; }
  const uint32_t* in_mask(int t) const {  // spike words of the input at step t (t >= 1)
    const uint32_t* base = graded() ? at<uint32_t>(lo.in_words) : reinterpret_cast<const uint32_t*>(in_base());
    return base + (size_t)(t - 1) * B * lo.words[0];
  }
  const float* in_dense(int t) const {   // graded input values at step t
    return reinterpret_cast<const float*>(in_base()) + (size_t)(t - 1) * B * net->sizes[0];
  }
  // Event arrays of the window in use: rows are addressed by the absolute step t, which must lie within the
  // window's segment, [ev_r0, ev_r0 + ev_steps + 1]; kernels that index by step get a base shifted accordingly.
  int ev_seg = 0, ev_r0 = 0;       // segment whose window the accessors address, and its first state
  size_t ev_shift = 0;             // byte offset of that window from the first one
  float* vals(int l) const { return at<float>(lo.vals[l] + ev_shift); }
  uint16_t* pref(int l, int t) const { return at<uint16_t>(lo.pref[l] + ev_shift) + ((ptrdiff_t)t - ev_r0) * B * lo.words[l]; }
  float* act(int l, int parity) const { return at<float>(lo.act[l]) + (size_t)parity * B * net->sizes[l]; }
  uint32_t* mask(int l, int t) const { return at<uint32_t>(lo.mask[l] + ev_shift) + ((ptrdiff_t)t - ev_r0) * B * lo.words[l]; }
  uint32_t* off(int l, int t) const { return at<uint32_t>(lo.off[l] + ev_shift) + ((ptrdiff_t)t - ev_r0) * B; }
  uint32_t* pool(int l) const { return at<uint32_t>(lo.pool[l] + ev_shift); }

  // ---- event windows (SNN_FLAG_SPILL_EVENTS)
  int ev_resident[2] = {0, -1};    // segment each window holds
  bool ev_pending[2] = {false, false};
  char* ev_host(int seg) const {
    return static_cast<char*>(a->pinned_ws) + (lo.tier2_on_device ? 0 : (size_t)lo.n_remote * lo.state_bytes) +
           (size_t)seg * lo.ev_window_bytes;
  }
  void ev_select(int seg) {
    ev_seg = seg; ev_r0 = seg * lo.ev_steps; ev_shift = (size_t)(seg & 1) * lo.ev_window_bytes;
    rows_params_ready = false;
  }
  // The main stream waits for the copy that last touched window w, if one is pending.
  snn_status ev_wait(int w) {
    if (ev_pending[w]) { CUDA_TRY(cudaStreamWaitEvent(main, net->ev_window[w], 0)); ev_pending[w] = false; }
    return SNN_OK;
  }
  // A copy of window w on the side stream, after everything issued so far on the main stream.
  snn_status ev_copy(int w, int seg, bool to_host) {
    if (!net->ev_window[w]) CUDA_TRY(cudaEventCreateWithFlags(&net->ev_window[w], cudaEventDisableTiming));   // once per net
    CUDA_TRY(cudaEventRecord(net->ev_main, main));
    CUDA_TRY(cudaStreamWaitEvent(side, net->ev_main, 0));
    char* dev = ws + lo.ev_base + (size_t)w * lo.ev_window_bytes;
    const int span = begin_span(to_host ? SNN_PHASE_D2H : SNN_PHASE_H2D, side);
    if (to_host) CUDA_TRY(cudaMemcpyAsync(ev_host(seg), dev, lo.ev_window_bytes, cudaMemcpyDeviceToHost, side));
    else CUDA_TRY(cudaMemcpyAsync(dev, ev_host(seg), lo.ev_window_bytes, cudaMemcpyHostToDevice, side));
    end_span(span, side);
    CUDA_TRY(cudaEventRecord(net->ev_window[w], side));
    ev_pending[w] = true;
    ++ev_copies;
    return SNN_OK;
  }
  int ev_copies = 0;
  // Forward pass enters segment seg (> 0): its window is free once the segment before the previous one has been
  // written out; the spike words of the boundary state come over from the previous window, list offsets restart.
  snn_status ev_enter_forward(int seg) {
    const int w = seg & 1, r0 = seg * lo.ev_steps;
    if (ev_wait(w) != SNN_OK) return SNN_ERR_CUDA;
    for (int l = 1; l <= L; ++l) {
      const uint32_t* src = mask(l, r0);   // still the previous segment's window: its last row
      uint32_t* dst = at<uint32_t>(lo.mask[l] + (size_t)w * lo.ev_window_bytes);
      CUDA_TRY(cudaMemcpyAsync(dst, src, 4 * (size_t)B * lo.words[l], cudaMemcpyDeviceToDevice, main));
    }
    for (int l = 0; l <= L; ++l)
      CUDA_TRY(cudaMemsetAsync(ws + lo.off[l] + (size_t)w * lo.ev_window_bytes, 0, 4 * (size_t)2 * B, main));
    ev_select(seg);
    ev_resident[w] = seg;
    return SNN_OK;
  }
  // Backward pass enters segment seg: its window must have arrived; the window of the segment after it is done
  // with and receives the segment before it.
  snn_status ev_enter_backward(int seg) {
    const int w = seg & 1;
    if (ev_resident[w] != seg) return fail(net, SNN_ERR_CUDA, "event window of segment %d is not resident", seg);
    if (ev_wait(w) != SNN_OK) return SNN_ERR_CUDA;
    ev_select(seg);
    if (seg >= 1 && ev_resident[w ^ 1] != seg - 1) {
      if (ev_wait(w ^ 1) != SNN_OK || ev_copy(w ^ 1, seg - 1, false) != SNN_OK) return SNN_ERR_CUDA;
      ev_resident[w ^ 1] = seg - 1;
    }
    return SNN_OK;
  }

  // The main stream waits for the checkpoint copy that last touched local slot s, if one is pending.
  snn_status wait_slot(int s) {
    if (!remote_tier || s < 0 || s >= (int)slot_event.size() || slot_event[s] < 0) return SNN_OK;
    const int e = slot_event[s];
    CUDA_TRY(cudaStreamWaitEvent(main, net->copy_events[e], 0));
    for (int& x : slot_event)
      if (x == e) x = -1;
    return SNN_OK;
  }

  void fill_fwd_layer(FwdLayer& f, int l, int t, const snn_op& op, bool gen) {
    const auto& sz = net->sizes;
    const int t0 = op.t0;
    f.mode = 1;
    f.W_ff = a->W_ff[l - 1];
    f.W_rec = a->W_rec[l - 1];
    f.N_pre = sz[l - 1]; f.N = sz[l]; f.W_pre = lo.words[l - 1]; f.W = lo.words[l];
    f.V_prev = t - 1 == t0 ? slot(op.in_slot, l) : slot(op.buf_slot + (t - 1 - t0 - 1) % op.buf_len, l);
    f.V_out = slot(op.buf_slot + (t - t0 - 1) % op.buf_len, l);
    f.V_keep = (op.keep_every > 0 && (t - t0) % op.keep_every == 0)
                   ? slot(op.keep_slot + (t - t0) / op.keep_every - 1, l) : nullptr;
    f.V_dbg = (gen && a->debug_V && a->debug_V[l - 1]) ? a->debug_V[l - 1] + (size_t)t * B * sz[l] : nullptr;
    f.ff_mask = l == 1 ? in_mask(t) : mask(l - 1, t);
    f.rec_mask = mask(l, t - 1);
    f.out_mask = mask(l, t);
    f.ff_pool = pool(l - 1); f.ff_off = off(l - 1, t); f.ff_cap = lo.cap[l - 1];
    f.rec_pool = pool(l); f.rec_off = off(l, t - 1); f.rec_cap = lo.cap[l];
    f.counts = (gen && l == L) ? at<uint32_t>(lo.counts) : nullptr;
    f.write_ff_list = l == 1;
    if (graded()) {
      f.ff_val_src = l == 1 ? in_dense(t) : act(l - 1, t & 1);
      f.rec_val_src = act(l, (t - 1) & 1);
      f.act_out = act(l, t & 1);
      f.ff_vals = vals(l - 1); f.rec_vals = vals(l);
      f.ff_pref = pref(l - 1, t); f.rec_pref = pref(l, t - 1);
    }
  }

  // Launch with programmatic stream serialization (the kernels call griddepcontrol.wait before they
  // touch global memory), optionally as thread-block clusters of cluster_x CTAs along x.
  template <class P> cudaError_t launch_pdl(void (*kernel)(P), dim3 grid, dim3 block, size_t smem, const P& params,
                                            int cluster_x = 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = main;
    cudaLaunchAttribute at[2];
    int n = 0;
    at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 0) {
      at[n].id = cudaLaunchAttributeClusterDimension;
      at[n].val.clusterDim.x = cluster_x; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
      ++n;
    }
    cfg.attrs = at; cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, params);
  }

  dim3 fwd_grid() const {
    int maxN = 0;
    for (int l = 1; l <= L; ++l) maxN = std::max(maxN, net->sizes[l]);
    return dim3((maxN + FWD_COLS - 1) / FWD_COLS, B, L);
  }

  snn_status launch_fwd(const FwdParams& p, bool gen) {
    void (*k)(FwdParams) = graded() ? (gen ? fwd_step_kernel<true, true> : fwd_step_kernel<false, true>)
                                    : (gen ? fwd_step_kernel<true, false> : fwd_step_kernel<false, false>);
    CUDA_TRY(launch_pdl(k, fwd_grid(), dim3(FWDS_THREADS), FWD_DYN_SMEM, p));
    ++launches;
    CUDA_TRY(cudaGetLastError());
    return SNN_OK;
  }

  // REFWD1 / REFWD2 without one launch per step: the stored events make the input current of every step
  // independent of the steps before it, so a run of steps is two launches, all currents at once and then
  // the leak/reset recurrence (refwd_gather_kernel, refwd_scan_kernel).  A run is as long as the ring of
  // state slots the operation writes to.  Used while the weights stay in L2; beyond that the per-step
  // launches keep the samples in step, and the rows they share are read from HBM once.
  bool reforward_runs_possible(const snn_op& op) const {
    if (a->flags & SNN_FLAG_REFORWARD_PER_STEP) return false;
    if (reforward_rows()) return true;
    if (!lo.weights_resident && !graded()) return false;
    return (long long)L * fwd_grid().x <= 65535 && std::min(op.buf_len, op.t1 - op.t0) <= 65535;
  }
  // the currents of a run come from refwd_rows_kernel (weight rows stationary) rather than refwd_gather_kernel
  // (spiking cell beyond L2 by default; the graded cell only on request: with values to fetch per event and 10 %
  // activity its rows-stationary pass measured slower than the per-step gather on the benchmark's graded network)
  bool reforward_rows() const {
    return (!lo.weights_resident && !graded()) || (a->flags & SNN_FLAG_REFORWARD_ROWS);
  }

  // tensor maps of the feed-forward matrices for ff_gemm_tc_kernel: 0 not tried yet, 1 ready, -1 not encodable
  CUtensorMap ffw_map[MAXL];
  int ffw_map_ready[MAXL] = {0};

  // Input currents of steps t0+d0+1 .. t0+d0+n with the weight rows stationary (weights beyond L2).
  RowsParams rows_params;        // tensor maps and per-layer constants, filled on first use in a step
  bool rows_params_ready = false;
  snn_status launch_reforward_rows(const snn_op& op, int d0, int n) {
    RowsParams& r = rows_params;
    int slabs_all = 0, slabs_max = 0, blocks_max = 0;
    for (int l = 1; l <= L; ++l) {
      const int slabs = (net->sizes[l] + RR_COLS - 1) / RR_COLS;
      slabs_all += slabs; slabs_max = std::max(slabs_max, slabs);
      blocks_max = std::max(blocks_max, lo.words[l - 1] + lo.words[l]);
    }
    // pairs per CTA: as many as a CTA can hold, halved while the grid would leave SMs without two CTAs
    // (every block of pairs streams the rows again; blocks of one slab are neighbours in launch order and
    // share the rows through L2)
    const int pairs = n * B;
    int pb = RR_MAX_PB;
    while (pb > 16 && (pb / 2 >= pairs || (long long)slabs_all * ((pairs + pb - 1) / pb) < 2 * 148)) pb /= 2;
    const int n_pb = (pairs + pb - 1) / pb;
    if (!rows_params_ready) {
      std::memset(&r, 0, sizeof r);
      size_t ev_off = 0;
      const size_t stride_max = lo.rows_ev_stride;
      for (int l = 1; l <= L; ++l) {
        RowsLayer& s = r.lay[l - 1];
        s.ff_words = l == 1 ? in_mask(1) : mask(l - 1, 0);
        s.ff_row0 = l == 1 ? 1 : 0;
        s.words = mask(l, 0);
        s.state_off = lo.layer_off[l];
        s.N_pre = net->sizes[l - 1]; s.N = net->sizes[l]; s.W_pre = lo.words[l - 1]; s.W = lo.words[l];
        s.ev_off = ev_off;
        ev_off += stride_max * ((size_t)s.W_pre + s.W);
        if (!make_tensor_map_2d(&r.map_ff[l - 1], a->W_ff[l - 1], (uint64_t)s.N_pre, (uint64_t)s.N, (uint64_t)s.N, RR_ROWS, RR_COLS, false) ||
            !make_tensor_map_2d(&r.map_rec[l - 1], a->W_rec[l - 1], (uint64_t)s.N, (uint64_t)s.N, (uint64_t)s.N, RR_ROWS, RR_COLS, false))
          return fail(net, SNN_ERR_CUDA, "tensor map of a weight matrix could not be encoded");
      }
      r.slots = at<float>(lo.slots); r.slot_stride = lo.state_bytes / 4;
      r.events = at<uint32_t>(lo.rows_ev); r.raw_off = lo.rows_ev_words;
      r.status = at<uint32_t>(lo.status);
      r.B = B;
      rows_params_ready = true;
    }
    r.t0 = op.t0; r.d0 = d0; r.n = n; r.buf_slot = op.buf_slot; r.buf_len = op.buf_len;
    r.pb = pb; r.ev_stride = n_pb * pb;
    if (graded()) {
      RowsGradedParams gp;
      std::memset(&gp, 0, sizeof gp);
      gp.r = r;
      gp.plane = lo.rows_ev_words;
      for (int l = 1; l <= L; ++l) {
        RowsGradedLayer& g = gp.g[l - 1];
        g.ff_off = off(l - 1, 0); g.ff_pref = pref(l - 1, 0); g.ff_vals = vals(l - 1); g.ff_cap = lo.cap[l - 1];
        g.rec_off = off(l, 0); g.rec_pref = pref(l, 0); g.rec_vals = vals(l); g.rec_cap = lo.cap[l];
      }
      CUDA_TRY(launch_pdl(rows_events_graded_kernel, dim3((unsigned)((r.ev_stride + 127) / 128), (unsigned)blocks_max, (unsigned)L),
                          dim3(128), 0, gp));
      CUDA_TRY(launch_pdl(refwd_rows_graded_kernel, dim3((unsigned)n_pb, (unsigned)slabs_max, (unsigned)L),
                          dim3(32 * (pb / RR_PPW + 1)), refwd_rows_graded_smem_bytes(pb), gp));
      launches += 2;
      return SNN_OK;
    }
    CUDA_TRY(launch_pdl(rows_events_kernel, dim3((unsigned)((r.ev_stride + 127) / 128), (unsigned)blocks_max, (unsigned)L),
                        dim3(128), 0, r));
    CUDA_TRY(launch_pdl(refwd_rows_kernel, dim3((unsigned)n_pb, (unsigned)slabs_max, (unsigned)L),
                        dim3(32 * (pb / RR_PPW + 1)), refwd_rows_smem_bytes(pb), r));
    launches += 2;
    return SNN_OK;
  }

  snn_status run_reforward_runs(const snn_op& op) {
    SegParams g;
    std::memset(&g, 0, sizeof g);
    g.slots = at<float>(lo.slots); g.slot_stride = lo.state_bytes / 4;
    g.B = B; g.t0 = op.t0; g.buf_slot = op.buf_slot; g.buf_len = op.buf_len;
    for (int l = 1; l <= L; ++l) {
      SegLayer& s = g.lay[l - 1];
      s.W_ff = a->W_ff[l - 1]; s.W_rec = a->W_rec[l - 1];
      s.ff_pool = pool(l - 1); s.ff_off = off(l - 1, 0); s.ff_cap = lo.cap[l - 1];
      s.rec_pool = pool(l); s.rec_off = off(l, 0); s.rec_cap = lo.cap[l];
      if (graded()) { s.ff_vals = vals(l - 1); s.rec_vals = vals(l); }
      s.state_off = lo.layer_off[l];
      s.N = net->sizes[l]; s.N_pre = net->sizes[l - 1];
    }
    g.status = at<uint32_t>(lo.status);
    ScanParams c;
    std::memset(&c, 0, sizeof c);
    c.slots = g.slots; c.slot_stride = g.slot_stride; c.n_quads = lo.state_bytes / 16;
    c.carry = at<float>(lo.vcarry);
    c.t0 = op.t0; c.buf_slot = op.buf_slot; c.buf_len = op.buf_len;
    c.keep_every = op.keep_every; c.keep_slot = op.keep_slot;
    c.alpha = net->alpha; c.theta = net->theta;
    void (*kg)(SegParams) = graded() ? refwd_gather_kernel<true> : refwd_gather_kernel<false>;
    void (*kc)(ScanParams) = graded() ? refwd_scan_kernel<true> : refwd_scan_kernel<false>;
    const int n_all = op.t1 - op.t0;
    const dim3 fg = fwd_grid();
    for (int d0 = 0; d0 < n_all; d0 += op.buf_len) {
      const int n = std::min(op.buf_len, n_all - d0);
      g.d0 = c.d0 = d0; g.n = c.n = n;
      c.v_start = d0 == 0 ? at<float>(lo.slots) + (size_t)op.in_slot * g.slot_stride : c.carry;
      if (!reforward_rows()) {
        g.tiles = (int)fg.x;
        CUDA_TRY(launch_pdl(kg, dim3((unsigned)B, (unsigned)n, (unsigned)L * fg.x), dim3(FWD_THREADS), REFWD_DYN_SMEM, g));
        ++launches;
      } else if (const snn_status st = launch_reforward_rows(op, d0, n); st != SNN_OK) {
        return st;
      }
      CUDA_TRY(launch_pdl(kc, dim3((unsigned)((c.n_quads + 127) / 128)), dim3(128), 0, c));
      ++launches;
    }
    CUDA_TRY(cudaGetLastError());
    return SNN_OK;
  }

  // FWD as one cooperative launch per op: CTAs wait for the spike words they need, sample by sample
  // (fwd_segment_kernel).  Possible when all CTAs of the grid are resident together.
  bool forward_segment_possible() {
    if (graded() || !lo.weights_resident || (a->flags & SNN_FLAG_FORWARD_PER_STEP)) return false;
    for (int l = 1; l <= L; ++l)
      if (lo.words[l - 1] + lo.words[l] > SEG_WORDS) return false;
    // CTAs the device holds at once with a deep copy ring ([0]: SEG_RING_MAX groups) and with a shallow one ([1])
    if (net->fwd_segment_capacity[0] < 0) {
      int dev = 0, sms = 0, coop = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) {
        cudaGetLastError();
        coop = 0;
      }
      for (int i = 0; i < 2; ++i) {
        int per_sm = 0;
        if (!coop || cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fwd_segment_kernel, FWDS_THREADS,
                                                                   (size_t)(i == 0 ? SEG_RING_MAX : GATHER_STAGES) * FWDS_GROUP_BYTES) != cudaSuccess) {
          cudaGetLastError();
          per_sm = 0;
        }
        net->fwd_segment_capacity[i] = sms * per_sm;
      }
    }
    const dim3 g = fwd_grid();
    return (long long)g.x * g.y * g.z <= std::max(net->fwd_segment_capacity[0], net->fwd_segment_capacity[1]);
  }

  // FWD with the weights held in shared memory for the whole launch (fwd_resident_kernel): small LIF networks.
  size_t resident_smem_max() const {
    size_t m = 0;
    for (int l = 1; l <= L; ++l)
      m = std::max(m, resident_smem_bytes(net->sizes[l - 1], net->sizes[l], lo.words[l - 1], lo.words[l], B));
    return m;
  }
  bool forward_resident_possible() {
    if (graded() || (a->flags & (SNN_FLAG_FORWARD_PER_STEP | SNN_FLAG_FORWARD_STREAM_WEIGHTS))) return false;
    if (B > 32 * RS_MAX_GROUPS) return false;
    long long ctas = 0;
    for (int l = 1; l <= L; ++l) {
      if (net->sizes[l - 1] + net->sizes[l] > 65535) return false;
      ctas += (net->sizes[l] + RS_COLS - 1) / RS_COLS;
    }
    const size_t smem = resident_smem_max();
    if (smem > RESIDENT_SMEM_MAX) return false;
    if (net->coop_sms < 0) {
      int dev = 0, sms = 0, coop = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) {
        cudaGetLastError();
        net->coop_sms = 0;
      } else {
        net->coop_sms = coop ? sms : 0;
      }
    }
    return ctas <= net->coop_sms;   // one CTA per SM (more than half of its shared memory each)
  }

  // `done` stays false when the device refuses the cooperative launch: the caller then takes the next path.
  snn_status run_forward_resident(const snn_op& op, bool& done) {
    done = false;
    ResParams p;
    std::memset(&p, 0, sizeof p);
    p.slots = at<float>(lo.slots); p.slot_stride = lo.state_bytes / 4;
    p.status = at<uint32_t>(lo.status); p.progress = at<uint32_t>(lo.progress);
    p.L = L; p.B = B; p.t0 = op.t0; p.t1 = op.t1;
    p.in_slot = op.in_slot; p.buf_slot = op.buf_slot; p.buf_len = op.buf_len;
    p.keep_every = op.keep_every; p.keep_slot = op.keep_slot;
    p.alpha = net->alpha; p.theta = net->theta;
    int ctas = 0;
    for (int l = 1; l <= L; ++l) {
      ResLayer& s = p.lay[l - 1];
      s.W_ff = a->W_ff[l - 1]; s.W_rec = a->W_rec[l - 1];
      s.ff_words = l == 1 ? in_mask(1) : mask(l - 1, 0);
      s.ff_row0 = l == 1 ? 1 : 0;
      s.words = mask(l, 0);
      s.ff_pool = pool(l - 1); s.ff_off = off(l - 1, 0); s.ff_cap = lo.cap[l - 1];
      s.rec_pool = pool(l); s.rec_off = off(l, 0); s.rec_cap = lo.cap[l];
      s.counts = l == L ? at<uint32_t>(lo.counts) : nullptr;
      s.V_dbg = (a->debug_V && a->debug_V[l - 1]) ? a->debug_V[l - 1] : nullptr;
      s.state_off = lo.layer_off[l];
      s.N_pre = net->sizes[l - 1]; s.N = net->sizes[l]; s.W_pre = lo.words[l - 1]; s.W = lo.words[l];
      s.write_ff_list = l == 1;
      s.tiles = (net->sizes[l] + RS_COLS - 1) / RS_COLS;
      s.cta0 = ctas;
      ctas += s.tiles;
    }
    const size_t smem = resident_smem_max();   // at most RESIDENT_SMEM_MAX, which the kernel is opted in for
    CUDA_TRY(cudaMemsetAsync(ws + lo.progress, 0, 4 * (size_t)L, main));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas); cfg.blockDim = dim3(RS_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = main;
    cudaLaunchAttribute at1[1];
    at1[0].id = cudaLaunchAttributeCooperative;
    at1[0].val.cooperative = 1;
    cfg.attrs = at1; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, fwd_resident_kernel, p) != cudaSuccess) {
      cudaGetLastError();
      return SNN_OK;
    }
    ++launches;
    done = true;
    return SNN_OK;
  }

  snn_status run_forward_segment(const snn_op& op, bool& done) {
    done = false;
    FwdSegParams p;
    std::memset(&p, 0, sizeof p);
    p.slots = at<float>(lo.slots); p.slot_stride = lo.state_bytes / 4;
    p.status = at<uint32_t>(lo.status); p.progress = at<uint32_t>(lo.progress);
    p.B = B; p.t0 = op.t0; p.t1 = op.t1;
    p.in_slot = op.in_slot; p.buf_slot = op.buf_slot; p.buf_len = op.buf_len;
    p.keep_every = op.keep_every; p.keep_slot = op.keep_slot;
    p.alpha = net->alpha; p.theta = net->theta;
    for (int l = 1; l <= L; ++l) {
      FwdSegLayer& s = p.lay[l - 1];
      s.W_ff = a->W_ff[l - 1]; s.W_rec = a->W_rec[l - 1];
      s.ff_words = l == 1 ? in_mask(1) : mask(l - 1, 0);
      s.ff_row0 = l == 1 ? 1 : 0;
      s.words = mask(l, 0);
      s.ff_pool = pool(l - 1); s.ff_off = off(l - 1, 0); s.ff_cap = lo.cap[l - 1];
      s.rec_pool = pool(l); s.rec_off = off(l, 0); s.rec_cap = lo.cap[l];
      s.counts = l == L ? at<uint32_t>(lo.counts) : nullptr;
      s.V_dbg = (a->debug_V && a->debug_V[l - 1]) ? a->debug_V[l - 1] : nullptr;
      s.state_off = lo.layer_off[l];
      s.N_pre = net->sizes[l - 1]; s.N = net->sizes[l]; s.W_pre = lo.words[l - 1]; s.W = lo.words[l];
      s.write_ff_list = l == 1;
      s.tiles = (net->sizes[l] + FWD_COLS - 1) / FWD_COLS;
    }
    CUDA_TRY(cudaMemsetAsync(ws + lo.progress, 0, 4 * (size_t)L * B, main));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = fwd_grid(); cfg.blockDim = dim3(FWDS_THREADS); cfg.stream = main;
    // the deep ring when the device holds the grid that way (one CTA per SM), else the shallow one
    p.ring_groups = (long long)cfg.gridDim.x * cfg.gridDim.y * cfg.gridDim.z <= net->fwd_segment_capacity[0] ? SEG_RING_MAX : GATHER_STAGES;
    cfg.dynamicSmemBytes = (size_t)p.ring_groups * FWDS_GROUP_BYTES;
    cudaLaunchAttribute at1[1];
    at1[0].id = cudaLaunchAttributeCooperative;
    at1[0].val.cooperative = 1;
    cfg.attrs = at1; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, fwd_segment_kernel, p) != cudaSuccess) {
      cudaGetLastError();
      return SNN_OK;
    }
    ++launches;
    done = true;
    return SNN_OK;
  }

  // FWD / REFWD1 / REFWD2: layer wavefront, layer l runs l-1 steps behind layer 1.
  snn_status run_forward(const snn_op& op, bool gen) {
    if (wait_slot(op.in_slot) != SNN_OK || wait_slot(op.keep_slot) != SNN_OK) return SNN_ERR_CUDA;
    const int n = op.t1 - op.t0;
    const int span = begin_span(op.kind == SNN_OP_FWD ? SNN_PHASE_FWD
                                : op.kind == SNN_OP_REFWD1 ? SNN_PHASE_REFWD1 : SNN_PHASE_REFWD2);
    if (!gen && reforward_runs_possible(op)) {
      const snn_status st = run_reforward_runs(op);
      end_span(span);
      return st;
    }
    if (gen && forward_resident_possible()) {
      bool done = false;
      const snn_status st = run_forward_resident(op, done);
      if (st != SNN_OK || done) { end_span(span); return st; }
    }
    if (gen && forward_segment_possible()) {
      bool done = false;
      const snn_status st = run_forward_segment(op, done);
      if (st != SNN_OK || done) { end_span(span); return st; }
    }
    FwdParams p;
    std::memset(&p, 0, sizeof p);
    p.B = B; p.alpha = net->alpha; p.theta = net->theta; p.status = at<uint32_t>(lo.status);
    for (int s = 1; s <= n + L - 1; ++s) {
      for (int l = 1; l <= L; ++l) {
        const int t = op.t0 + s - (l - 1);
        if (t <= op.t0 || t > op.t1) p.lay[l - 1].mode = 0;
        else fill_fwd_layer(p.lay[l - 1], l, t, op, gen);
      }
      if (launch_fwd(p, gen) != SNN_OK) return SNN_ERR_CUDA;
    }
    end_span(span);
    return SNN_OK;
  }

  // After the last forward step (of the sequence, or of an event window): store the event lists of its spikes.
  snn_status run_flush(int t_end) {
    FwdParams p;
    std::memset(&p, 0, sizeof p);
    p.B = B; p.alpha = net->alpha; p.theta = net->theta; p.status = at<uint32_t>(lo.status);
    for (int l = 1; l <= L; ++l) {
      FwdLayer& f = p.lay[l - 1];
      f.mode = 2; f.N = net->sizes[l]; f.W = lo.words[l];
      f.rec_mask = mask(l, t_end); f.rec_pool = pool(l); f.rec_off = off(l, t_end); f.rec_cap = lo.cap[l];
      if (graded()) { f.rec_val_src = act(l, t_end & 1); f.rec_vals = vals(l); f.rec_pref = pref(l, t_end); }
    }
    return launch_fwd(p, true);
  }

  snn_status run_readout() {
    const int N_L = net->sizes[L], N_out = net->sizes[L + 1];
    const uint32_t* counts = at<uint32_t>(lo.counts);
    const int32_t* targets = (a->flags & SNN_FLAG_INPUT_ON_HOST) ? at<int32_t>(lo.tg_stage) : a->targets;
    const int span = begin_span(SNN_PHASE_READOUT);
    const int cf = graded() ? 1 : 0;
    readout_logits_kernel<<<B, 256, 8 * N_out * sizeof(float), main>>>(counts, cf, a->W_out, N_L, N_out, net->scale,
                                                                       at<float>(lo.logits));
    softmax_loss_kernel<<<1, 256, B * sizeof(float), main>>>(at<float>(lo.logits), targets, B, N_out,
                                                             at<float>(lo.dlogits), at<float>(lo.status) + 1,
                                                             at<uint32_t>(lo.status));
    launches += 2;
    if (!(a->flags & SNN_FLAG_FORWARD_ONLY)) {
      readout_gout_kernel<<<(unsigned)(((size_t)B * N_L + 255) / 256), 256, 0, main>>>(
          a->W_out, at<float>(lo.dlogits), B, N_L, N_out, net->scale, at<float>(lo.g_out));
      readout_dwout_kernel<<<(unsigned)(((size_t)N_L * N_out + 255) / 256), 256, 0, main>>>(
          counts, cf, at<float>(lo.dlogits), B, N_L, N_out, net->scale, a->dW_out);
      launches += 2;
    }
    end_span(span);
    CUDA_TRY(cudaGetLastError());
    return SNN_OK;
  }

  template <int U> void launch_dw(DwParams& d, int maxN, int maxNpre) {
    dim3 grid((maxN + 128 * U - 1) / (128 * U), (maxNpre + DW_ROWS - 1) / DW_ROWS, 2 * L);
    const int pairs = d.n_steps * d.B;
    d.window = std::min(DW_WINDOW, (pairs + 31) / 32 * 32);
    if (graded()) launch_pdl(dw_kernel<U, true>, grid, dim3(32 * DW_ROWS), dw_smem_bytes<U, true>(d.window), d);
    else launch_pdl(dw_kernel<U, false>, grid, dim3(32 * DW_ROWS), dw_smem_bytes<U, false>(d.window), d);
    ++launches;
  }
  // dynamic shared memory of bwd_step_kernel for BP samples per pass: the staged tiles
  static size_t bwd_smem_bytes(int bp, int ld = BWD_LD) { return (size_t)BWD_STAGES * (BWD_TM + bp) * ld * sizeof(float); }
  template <int NTN, int NWARP> cudaError_t launch_bwd(const BwdParams& p, int tiles, int CS, int n_layers = 0) {
    return launch_pdl(bwd_step_kernel<NTN, NWARP>, dim3(tiles * CS, 1, n_layers ? n_layers : L), dim3(32 * NWARP),
                      bwd_smem_bytes(8 * NTN, bwd_ld(NWARP)), p, CS);
  }

  // BWD: layer wavefront, layer l runs L-l steps behind the last layer; then the weight
  // gradients of the whole segment.
  // BWD as one cooperative launch of thread-block clusters (bwd_segment_kernel), if every CTA's slice of the
  // weights fits in shared memory and the device can hold all clusters at once; otherwise `done` stays false.
  template <int NTN, int NWARP> snn_status try_backward_segment(const snn_op& op, int CS, bool& done) {
    const auto& sz = net->sizes;
    done = false;
    BwdSegParams p;
    std::memset(&p, 0, sizeof p);
    size_t res_floats = 0;
    int ctas = 0;
    for (int l = 1; l <= L; ++l) {
      BwdSegLayer& f = p.lay[l - 1];
      f.N = sz[l]; f.N_post = l < L ? sz[l + 1] : 0;
      f.W_rec = a->W_rec[l - 1];
      f.W_ffa = l < L ? a->W_ff[l] : nullptr;
      f.g_out = l == L ? at<float>(lo.g_out) : nullptr;
      f.carry_in = carry(carry_cur, l);
      f.carry_out = carry(carry_cur ^ 1, l);
      f.state_off = lo.layer_off[l];
      f.state_off_above = l < L ? lo.layer_off[l + 1] : 0;
      f.ctas = (sz[l] + BWD_TM - 1) / BWD_TM * CS;
      f.cta0 = ctas;
      ctas += f.ctas;
      const int q_rec = f.N / 4, q_ff = f.N_post / 4;
      for (int r = 0; r < CS; ++r) {
        const int k_rec = (int)((long long)q_rec * (r + 1) / CS) * 4 - (int)((long long)q_rec * r / CS) * 4;
        const int k_ff = (int)((long long)q_ff * (r + 1) / CS) * 4 - (int)((long long)q_ff * r / CS) * 4;
        res_floats = std::max(res_floats, (size_t)BWD_TM * bwd_resident_ld(k_ff, k_rec, NWARP));
      }
    }
    const size_t smem = 4 * (res_floats + bwd_segment_region_floats<NTN, NWARP>());
    if (smem > BWD_SEGMENT_SMEM_MAX) return SNN_OK;
    void (*k)(BwdSegParams) = bwd_segment_kernel<NTN, NWARP>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas); cfg.blockDim = dim3(32 * NWARP); cfg.dynamicSmemBytes = smem; cfg.stream = main;
    cudaLaunchAttribute at2[2];
    at2[0].id = cudaLaunchAttributeCooperative; at2[0].val.cooperative = 1;
    at2[1].id = cudaLaunchAttributeClusterDimension;
    at2[1].val.clusterDim.x = CS; at2[1].val.clusterDim.y = 1; at2[1].val.clusterDim.z = 1;
    cfg.attrs = at2; cfg.numAttrs = 2;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      cudaGetLastError();
      return SNN_OK;
    }
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, k, &cfg) != cudaSuccess || (long long)clusters * CS < ctas) {
      cudaGetLastError();
      return SNN_OK;
    }
    p.slots = at<float>(lo.slots); p.slot_stride = lo.state_bytes / 4;
    p.status = at<uint32_t>(lo.status); p.progress = at<uint32_t>(lo.progress);
    p.L = L; p.B = B; p.t0 = op.t0; p.t1 = op.t1; p.buf_slot = op.buf_slot;
    p.alpha = net->alpha; p.theta = net->theta; p.beta = net->beta;
    p.surrogate = net->surrogate; p.cell = net->cell;
    CUDA_TRY(cudaMemsetAsync(ws + lo.progress, 0, 4 * (size_t)L, main));
    if (cudaLaunchKernelEx(&cfg, k, p) != cudaSuccess) {   // e.g. refused under a profiler: one launch per step instead
      cudaGetLastError();
      return SNN_OK;
    }
    ++launches;
    done = true;
    return SNN_OK;
  }

  // Steps ts_hi-1 .. ts_lo of one layer in one cooperative launch (bwd_stream_kernel), if the device holds all
  // its CTAs at once; otherwise `done` stays false and the caller launches step by step.
  CUtensorMap wrec_map[MAXL];      // W_rec of a layer as boxes of 16 MT rows x 32 values: 0 not tried yet, 1 ready, -1 not encodable
  int wrec_map_ready[MAXL] = {0};
  template <int NTN, int NWARP, int MT> snn_status try_backward_stream(BwdStreamParams& sp, int l, int tiles, bool& done) {
    done = false;
    void (*k)(BwdStreamParams) = bwd_stream_kernel<NTN, NWARP, MT>;
    const size_t smem = bwd_stream_smem_bytes<NTN, NWARP, MT>();
    // tensor maps: the matrix once per step of the executor, the deltas of this run (strides must be multiples of 16 bytes)
    if (sp.N % 4 != 0 || sp.slot_stride % 4 != 0) return SNN_OK;
    sp.one_copy = sp.N % 32 == 0;
    if (wrec_map_ready[l - 1] == 0) {
      if (sp.one_copy) {
        const uint64_t dims[3] = {32, (uint64_t)sp.N, (uint64_t)sp.N / 32}, strides[2] = {(uint64_t)sp.N, 32};
        const uint32_t box[3] = {32, 16 * MT, 4};
        wrec_map_ready[l - 1] = make_tensor_map_nd(&wrec_map[l - 1], a->W_rec[l - 1], 3, dims, strides, box) ? 1 : -1;
      } else {
        wrec_map_ready[l - 1] = make_tensor_map_2d(&wrec_map[l - 1], a->W_rec[l - 1], (uint64_t)sp.N, (uint64_t)sp.N, (uint64_t)sp.N,
                                                   16 * MT, 32, true) ? 1 : -1;
      }
    }
    if (wrec_map_ready[l - 1] < 0) return SNN_OK;
    sp.map_w = wrec_map[l - 1];
    const float* const d_slots = sp.slots + (size_t)sp.buf_slot * sp.slot_stride + sp.state_off;
    if (sp.one_copy) {
      const uint64_t dims[4] = {32, (uint64_t)sp.B, (uint64_t)sp.N / 32, (uint64_t)sp.ts_hi}, dims0[4] = {32, (uint64_t)sp.B, (uint64_t)sp.N / 32, 1};
      const uint64_t strides[3] = {(uint64_t)sp.N, 32, (uint64_t)sp.slot_stride};
      const uint32_t box[4] = {32, 8 * NTN, 4, 1};
      if (!make_tensor_map_nd(&sp.map_d, d_slots, 4, dims, strides, box) || !make_tensor_map_nd(&sp.map_d0, sp.d_first, 4, dims0, strides, box))
        return SNN_OK;
    } else if (!make_tensor_map_3d(&sp.map_d, d_slots, (uint64_t)sp.N, (uint64_t)sp.B, (uint64_t)sp.ts_hi, (uint64_t)sp.N,
                                   (uint64_t)sp.slot_stride, 32, 8 * NTN, 1) ||
               !make_tensor_map_3d(&sp.map_d0, sp.d_first, (uint64_t)sp.N, (uint64_t)sp.B, 1, (uint64_t)sp.N, (uint64_t)sp.slot_stride, 32,
                                   8 * NTN, 1)) {
      return SNN_OK;
    }
    int& cap = net->bwd_stream_capacity[(NTN == 1 ? 0 : NTN == 2 ? 1 : 2) + 3 * (MT - 1)];
    if (cap < 0) {
      int dev = 0, sms = 0, per_sm = 0, coop = 0;
      if (cudaGetDevice(&dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
          cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess ||
          cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, 32 * (NWARP + 2), smem) != cudaSuccess) {
        cudaGetLastError();
        cap = 0;
      } else {
        cap = coop ? sms * per_sm : 0;
      }
    }
    if (tiles > cap) return SNN_OK;
    CUDA_TRY(cudaMemsetAsync(ws + lo.progress, 0, 4, main));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tiles); cfg.blockDim = dim3(32 * (NWARP + 2)); cfg.dynamicSmemBytes = smem; cfg.stream = main;
    cudaLaunchAttribute at1[1];
    at1[0].id = cudaLaunchAttributeCooperative;
    at1[0].val.cooperative = 1;
    cfg.attrs = at1; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, k, sp) != cudaSuccess) {
      cudaGetLastError();
      return SNN_OK;
    }
    ++launches;
    done = true;
    return SNN_OK;
  }

  snn_status run_backward(const snn_op& op) {
    const auto& sz = net->sizes;
    const int n = op.t1 - op.t0;
    BwdParams p;
    std::memset(&p, 0, sizeof p);
    p.B = B; p.alpha = net->alpha; p.theta = net->theta; p.beta = net->beta;
    p.surrogate = net->surrogate; p.cell = net->cell;
    int maxN = 0;
    for (int l = 1; l <= L; ++l) maxN = std::max(maxN, sz[l]);
    // cluster size along the contraction index: enough CTAs to fill the GPU, at least one full
    // warp pass (128 values) per rank; a function of the network sizes only
    const int tiles = (maxN + BWD_TM - 1) / BWD_TM;
    int minN = maxN;
    for (int l = 1; l <= L; ++l) minN = std::min(minN, sz[l]);
    // (one wave: two 256-thread CTAs or one 512-thread CTA per SM on 148 SMs)
    const int wave = B <= 16 ? 296 : 148;
    const int CS = backward_cluster_size(sz, L, B);
    int span = begin_span(SNN_PHASE_BWD);
    // event-driven steps (compact-support surrogate): a layer wavefront, one launch per step
    const bool event_driven = (a->flags & SNN_FLAG_BACKWARD_EVENT_DRIVEN) != 0;
    const bool layer_major = !event_driven && L > 1 && ((a->flags & SNN_FLAG_BACKWARD_LAYER_BY_LAYER) ||
                                       (lo.layer_major && !(a->flags & SNN_FLAG_BACKWARD_WAVEFRONT)));
    bool segment_done = false;
    if (!layer_major && !event_driven && !(a->flags & SNN_FLAG_BACKWARD_PER_STEP)) {
      // small networks: the whole segment in one cooperative launch, the weights resident in shared memory
      snn_status st = SNN_OK;
      if (B <= 8) st = try_backward_segment<1, 8>(op, CS, segment_done);
      else if (B <= 16) st = try_backward_segment<2, 8>(op, CS, segment_done);
      else st = try_backward_segment<4, 16>(op, CS, segment_done);
      if (st != SNN_OK) return st;
    }
    if (segment_done) {
    } else if (layer_major) {
      // Runs of at most BWD_RUN steps, latest first; within a run the layers go from the last to the first:
      // the feed-forward term of layer l for the whole run is one product (ff_gemm_kernel), then the steps
      // of layer l follow one launch each.
      int gff_parts = 1;   // partial products the feed-forward term of the current layer and run consists of
      for (int hi = n; hi > 0; hi -= BWD_RUN) {
        const int lo_s = std::max(0, hi - BWD_RUN);     // steps t0+lo_s+1 .. t0+hi
        for (int l = L; l >= 1; --l) {
          if (l < L) {
            end_span(span);
            span = begin_span(SNN_PHASE_FFGEMM);
            const int n_run = hi - lo_s;
            bool on_tcgen05 = false;
            gff_parts = 1;
            if (!(a->flags & SNN_FLAG_FF_PRODUCT_MMA_SYNC) && B <= TCG_NMAX) {
              // tcgen05 path: 128 rows of W x up to 128 pairs per CTA, accumulator in tensor memory
              TcGemmParams tp;
              std::memset(&tp, 0, sizeof tp);
              tp.steps_per_tile = std::min(n_run, TCG_NMAX / B);
              tp.n_cols = (tp.steps_per_tile * B + 15) / 16 * 16;
              tp.out = at<float>(lo.gff); tp.status = at<uint32_t>(lo.status);
              // few row tiles: the contraction range is cut into slices so that most SMs get a CTA; a function of
              // the layer width alone (partial products are added in slice order by the step kernel)
              const int row_tiles = (sz[l] + TCG_M - 1) / TCG_M;
              tp.k_split = std::max(1, std::min({TCG_MAX_KSPLIT, 148 / row_tiles, (sz[l + 1] + TCG_KB - 1) / TCG_KB}));
              tp.out_stride = lo.gff_stride;
              gff_parts = tp.k_split;
              tp.N = sz[l]; tp.K = sz[l + 1]; tp.B = B; tp.n_steps = n_run;
              if (!ffw_map_ready[l]) {
                ffw_map_ready[l] = make_tensor_map_2d(&ffw_map[l], a->W_ff[l], (uint64_t)sz[l], (uint64_t)sz[l + 1],
                                                      (uint64_t)sz[l + 1], TCG_M, TCG_KB, true) ? 1 : -1;
              }
              if (ffw_map_ready[l] > 0 &&
                  make_tensor_map_delta(&tp.map_d, slot(op.buf_slot + lo_s, l + 1), (uint64_t)sz[l + 1], (uint64_t)B,
                                        (uint64_t)n_run, lo.state_bytes / 4, (uint32_t)tp.steps_per_tile)) {
                tp.map_w = ffw_map[l];
                CUDA_TRY(launch_pdl(ff_gemm_tc_kernel,
                                    dim3((unsigned)((n_run + tp.steps_per_tile - 1) / tp.steps_per_tile),
                                         (unsigned)row_tiles, (unsigned)tp.k_split),
                                    dim3(TCG_THREADS), TCG_SMEM_BYTES, tp));
                on_tcgen05 = true;
              }
            }
            if (!on_tcgen05) {
              FfGemmParams gp;
              gp.W = a->W_ff[l]; gp.N = sz[l]; gp.K = sz[l + 1]; gp.B = B; gp.n_steps = n_run;
              gp.delta0 = slot(op.buf_slot + lo_s, l + 1); gp.slot_stride = lo.state_bytes / 4;
              gp.out = at<float>(lo.gff);
              CUDA_TRY(launch_pdl(ff_gemm_kernel, dim3((gp.n_steps * B + 8 * FFG_NTN - 1) / (8 * FFG_NTN), (sz[l] + BWD_TM - 1) / BWD_TM),
                                  dim3(32 * FFG_NWARP),
                                  bwd_smem_bytes(8 * FFG_NTN), gp));
            }
            ++launches;
            end_span(span);
            span = begin_span(SNN_PHASE_BWD);
          }
          const int tiles_l = (sz[l] + BWD_TM - 1) / BWD_TM;
          int CS_l = 1;
          // layers with a tile of 16 rows for every SM: no cluster, so that the run can be one launch that keeps the
          // weight stream going (bwd_stream_kernel; tiles of 32 rows where those still cover the SMs)
          const int tiles16_l = (sz[l] + 15) / 16;
          const bool wide = tiles_l >= 148 || (tiles16_l >= 148 && B <= 16);   // (two CTAs of 16 rows per SM need B <= 16)
          while (!wide && CS_l < 8 && tiles_l * CS_l * 2 <= wave && sz[l] / (4 * CS_l * 2) >= 32) CS_l *= 2;
          if (CS_l == 1 && B <= 32 && !(a->flags & SNN_FLAG_BACKWARD_PER_STEP)) {
            BwdStreamParams sp;
            std::memset(&sp, 0, sizeof sp);
            sp.g_out = l == L ? at<float>(lo.g_out) : nullptr;
            sp.g_ff = l < L ? at<float>(lo.gff) : nullptr;
            sp.g_ff_parts = gff_parts; sp.g_ff_stride = lo.gff_stride;
            sp.d_first = op.t0 + hi == op.t1 ? carry(carry_cur, l) : slot(op.buf_slot + hi, l);
            sp.carry_out = lo_s == 0 ? carry(carry_cur ^ 1, l) : nullptr;
            sp.slots = at<float>(lo.slots); sp.slot_stride = lo.state_bytes / 4; sp.state_off = lo.layer_off[l];
            sp.status = at<uint32_t>(lo.status); sp.progress = at<uint32_t>(lo.progress);
            sp.N = sz[l]; sp.B = B; sp.buf_slot = op.buf_slot; sp.ts_lo = lo_s; sp.ts_hi = hi;
            // part of W_rec asked to stay in L2 from one step to the next: whole chunks of 128 columns
            sp.keep_chunks = (int)std::min<size_t>((size_t)(sz[l] + 127) / 128, BWD_STREAM_KEEP_BYTES / ((size_t)sz[l] * 512));
            sp.alpha = net->alpha; sp.theta = net->theta; sp.beta = net->beta;
            sp.surrogate = net->surrogate; sp.cell = net->cell;
            bool done = false;
            snn_status st = SNN_OK;
            if (tiles_l >= 148) {
              if (B <= 8) st = try_backward_stream<1, 8, 2>(sp, l, tiles_l, done);
              else if (B <= 16) st = try_backward_stream<2, 8, 2>(sp, l, tiles_l, done);
              else st = try_backward_stream<4, 16, 2>(sp, l, tiles_l, done);
            } else {
              if (B <= 8) st = try_backward_stream<1, 8, 1>(sp, l, tiles16_l, done);
              else if (B <= 16) st = try_backward_stream<2, 8, 1>(sp, l, tiles16_l, done);
              else st = try_backward_stream<4, 16, 1>(sp, l, tiles16_l, done);
            }
            if (st != SNN_OK) return st;
            if (done) continue;
          }
          for (int ts = hi - 1; ts >= lo_s; --ts) {
            const int t = op.t0 + ts + 1;
            std::memset(&p.lay[0], 0, sizeof p.lay[0]);
            BwdLayer& f = p.lay[0];
            f.mode = 1;
            f.N = sz[l]; f.N_post = 0;
            f.W_rec = a->W_rec[l - 1];
            f.V_delta = slot(op.buf_slot + ts, l);
            f.d_next = t == op.t1 ? carry(carry_cur, l) : slot(op.buf_slot + ts + 1, l);
            f.g_out = l == L ? at<float>(lo.g_out) : nullptr;
            f.g_ff = l < L ? at<float>(lo.gff) + (size_t)(ts - lo_s) * B * sz[l] : nullptr;
            f.g_ff_parts = gff_parts; f.g_ff_stride = lo.gff_stride;
            f.carry_out = t == op.t0 + 1 ? carry(carry_cur ^ 1, l) : nullptr;
            cudaError_t le;
            if (B <= 8) le = launch_bwd<1, 8>(p, tiles_l, CS_l, 1);
            else if (B <= 16) le = launch_bwd<2, 8>(p, tiles_l, CS_l, 1);
            else le = launch_bwd<4, 16>(p, tiles_l, CS_l, 1);
            if (le != cudaSuccess) return fail(net, SNN_ERR_CUDA, "backward launch failed: %s", cudaGetErrorString(le));
            ++launches;
          }
        }
      }
    } else
    for (int s = 0; s <= n + L - 2; ++s) {
      for (int l = L; l >= 1; --l) {
        BwdLayer& f = p.lay[l - 1];
        const int lag = L - l, t = op.t1 - (s - lag);
        if (s < lag || t <= op.t0) { f.mode = 0; continue; }
        f.mode = 1;
        f.N = sz[l]; f.N_post = l < L ? sz[l + 1] : 0;
        f.W_rec = a->W_rec[l - 1];
        f.W_ffa = l < L ? a->W_ff[l] : nullptr;
        f.V_delta = slot(op.buf_slot + (t - op.t0 - 1), l);
        f.d_next = t == op.t1 ? carry(carry_cur, l) : slot(op.buf_slot + (t - op.t0), l);
        f.d_above = l < L ? slot(op.buf_slot + (t - op.t0 - 1), l + 1) : nullptr;
        f.g_out = l == L ? at<float>(lo.g_out) : nullptr;
        f.carry_out = t == op.t0 + 1 ? carry(carry_cur ^ 1, l) : nullptr;
      }
      cudaError_t le;
      if (event_driven) {
        const long long warps = (long long)((maxN + 31) / 32) * B;
        le = launch_pdl(bwd_event_kernel, dim3((unsigned)((warps + BEV_WARPS - 1) / BEV_WARPS), 1, (unsigned)L),
                        dim3(32 * BEV_WARPS), 0, p);
      }
      else if (B <= 8) le = launch_bwd<1, 8>(p, tiles, CS);
      else if (B <= 16) le = launch_bwd<2, 8>(p, tiles, CS);
      else le = launch_bwd<4, 16>(p, tiles, CS);
      if (le != cudaSuccess) return fail(net, SNN_ERR_CUDA, "backward launch failed: %s", cudaGetErrorString(le));
      ++launches;
    }
    carry_cur ^= 1;
    end_span(span);
    span = begin_span(SNN_PHASE_DW);
    // All 2L weight gradients of the segment in one launch.  Row positions are kept in units of 16 bytes in
    // 32 bits, so a very long segment (STANDARD) is cut into runs of steps, latest steps first: the order of
    // additions per element (t descending, b ascending) is unchanged.
    const size_t stride16 = lo.state_bytes / 16;
    const int max_run = (int)std::min<size_t>((size_t)n, (0xffffffffull - (size_t)B * maxN / 4) / stride16);
    int maxNpre = sz[0];
    for (int l = 1; l <= L; ++l) maxNpre = std::max(maxNpre, sz[l]);
    for (int hi = n; hi > 0; hi -= max_run) {
      const int lo_s = std::max(0, hi - max_run);   // steps t0+lo_s+1 .. t0+hi
      const int ta = op.t0 + lo_s;
      DwParams d;
      std::memset(&d, 0, sizeof d);
      d.B = B; d.n_steps = hi - lo_s; d.slot_stride = lo.state_bytes / 4;
      for (int l = 1; l <= L; ++l) {
        DwArgs& f = d.m[2 * (l - 1)];
        f.N = sz[l]; f.delta0 = slot(op.buf_slot + lo_s, l);
        f.dW = a->dW_ff[l - 1]; f.N_pre = sz[l - 1]; f.Wm = lo.words[l - 1];
        f.mask_row0 = l == 1 ? in_mask(ta + 1) : mask(l - 1, ta + 1);
        if (graded()) { f.off_row0 = off(l - 1, ta + 1); f.pref_row0 = pref(l - 1, ta + 1); f.vals = vals(l - 1); f.cap = lo.cap[l - 1]; }
        DwArgs& r = d.m[2 * (l - 1) + 1];
        r.N = sz[l]; r.delta0 = f.delta0;
        r.dW = a->dW_rec[l - 1]; r.N_pre = sz[l]; r.Wm = lo.words[l];
        r.mask_row0 = mask(l, ta);
        if (graded()) { r.off_row0 = off(l, ta); r.pref_row0 = pref(l, ta); r.vals = vals(l); r.cap = lo.cap[l]; }
      }
      const bool slab = !(a->flags & SNN_FLAG_WEIGHT_GRADIENT_GATHER) &&
                        (!lo.weights_resident || (a->flags & SNN_FLAG_WEIGHT_GRADIENT_SLAB));
      if (slab) {
        // the deltas stationary in shared memory, the rows of dW streamed past them (dw_slab_kernel)
        // rows per CTA: as many as amortise the copy of the slab, fewer while the grid would not fill the device four
        // times over (a function of the network alone)
        const long long slabs = (maxN + DWS_COLS - 1) / DWS_COLS;
        long long row_units = 0;
        d.slab_rows = DWS_ROWS;
        for (;;) {
          row_units = 0;
          for (int l = 1; l <= L; ++l)
            row_units += (sz[l - 1] + d.slab_rows - 1) / d.slab_rows + (sz[l] + d.slab_rows - 1) / d.slab_rows;
          if (d.slab_rows <= 256 || slabs * row_units >= 4 * 148) break;
          d.slab_rows /= 2;
        }
        const dim3 grid((unsigned)slabs, (unsigned)((maxNpre + d.slab_rows - 1) / d.slab_rows), 2u * L);
        if (graded()) launch_pdl(dw_slab_kernel<true>, grid, dim3(32 * DWS_WARPS), dws_smem_bytes<true>(), d);
        else launch_pdl(dw_slab_kernel<false>, grid, dim3(32 * DWS_WARPS), dws_smem_bytes<false>(), d);
        ++launches;
      }
      // wider column tiles for wider layers: the per-CTA compaction of the pair lists is amortised over more columns
      else if (maxN >= 1024) launch_dw<8>(d, maxN, maxNpre);
      else if (maxN >= 512) launch_dw<4>(d, maxN, maxNpre);
      else if (maxN >= 256) launch_dw<2>(d, maxN, maxNpre);
      else launch_dw<1>(d, maxN, maxNpre);
    }
    end_span(span);
    CUDA_TRY(cudaGetLastError());
    return SNN_OK;
  }

  snn_status run_copy(const snn_op& op) {
    const int count = std::max(1, op.buf_len);
    const size_t bytes = (size_t)count * lo.state_bytes;
    char* remote = (lo.tier2_on_device ? ws + lo.tier2 : static_cast<char*>(a->pinned_ws)) +
                   (size_t)op.remote_slot * lo.state_bytes;
    const bool out = op.kind == SNN_OP_D2H;
    const int s = out ? op.in_slot : op.keep_slot;
    char* local = ws + lo.slots + (size_t)s * lo.state_bytes;
    // a slot that an earlier copy still uses: order the two copies through the main stream
    for (int k = 0; k < count; ++k)
      if (wait_slot(s + k) != SNN_OK) return SNN_ERR_CUDA;
    // the copy starts after everything issued so far on the main stream
    CUDA_TRY(cudaEventRecord(net->ev_main, main));
    CUDA_TRY(cudaStreamWaitEvent(side, net->ev_main, 0));
    const int span = begin_span(out ? SNN_PHASE_D2H : SNN_PHASE_H2D, side);
    const cudaMemcpyKind kind = lo.tier2_on_device ? cudaMemcpyDeviceToDevice
                                                    : (out ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice);
    if (out) { CUDA_TRY(cudaMemcpyAsync(remote, local, bytes, kind, side)); ++d2h; }
    else { CUDA_TRY(cudaMemcpyAsync(local, remote, bytes, kind, side)); ++h2d; }
    end_span(span, side);
    // one event per copy in flight; events are reused once every slot that waited on them was released
    int e = 0;
    for (;; ++e) {
      bool used = false;
      for (int x : slot_event) used |= x == e;
      if (!used) break;
    }
    while ((int)net->copy_events.size() <= e) {
      cudaEvent_t ev;
      CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
      net->copy_events.push_back(ev);
    }
    CUDA_TRY(cudaEventRecord(net->copy_events[e], side));
    for (int k = 0; k < count; ++k) slot_event[s + k] = e;
    return SNN_OK;
  }
};

}  // namespace

namespace {
// Kernels that use more than 48 KB of dynamic shared memory are opted in once per device (the attribute belongs
// to the function on one device); a mutex orders host threads that take their first step at the same time.
constexpr int kMaxDevices = 64;
std::mutex g_device_mutex;
bool g_smem_opted_in[kMaxDevices] = {false};

snn_status opt_in_shared_memory(snn_net* net, int dev) {
  if (dev < 0 || dev >= kMaxDevices) return fail(net, SNN_ERR_UNSUPPORTED, "device index %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (g_smem_opted_in[dev]) return SNN_OK;
  const auto dyn = cudaFuncAttributeMaxDynamicSharedMemorySize;
  CUDA_TRY(cudaFuncSetAttribute(fwd_step_kernel<true, false>, dyn, (int)FWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(fwd_step_kernel<false, false>, dyn, (int)FWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(fwd_step_kernel<true, true>, dyn, (int)FWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(fwd_step_kernel<false, true>, dyn, (int)FWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(fwd_segment_kernel, dyn, (int)(SEG_RING_MAX * FWDS_GROUP_BYTES)));
  CUDA_TRY(cudaFuncSetAttribute(fwd_resident_kernel, dyn, (int)RESIDENT_SMEM_MAX));
  CUDA_TRY(cudaFuncSetAttribute(refwd_gather_kernel<false>, dyn, (int)REFWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(refwd_gather_kernel<true>, dyn, (int)REFWD_DYN_SMEM));
  CUDA_TRY(cudaFuncSetAttribute(refwd_rows_kernel, dyn, (int)refwd_rows_smem_bytes(RR_MAX_PB)));
  CUDA_TRY(cudaFuncSetAttribute(refwd_rows_graded_kernel, dyn, (int)refwd_rows_graded_smem_bytes(RR_MAX_PB)));
  CUDA_TRY(cudaFuncSetAttribute(ff_gemm_kernel, dyn, (int)Exec::bwd_smem_bytes(8 * FFG_NTN)));
  CUDA_TRY(cudaFuncSetAttribute(ff_gemm_tc_kernel, dyn, (int)TCG_SMEM_BYTES));
  CUDA_TRY(cudaFuncSetAttribute(bwd_step_kernel<1, 8>, dyn, (int)Exec::bwd_smem_bytes(8, bwd_ld(8))));
  CUDA_TRY(cudaFuncSetAttribute(bwd_step_kernel<2, 8>, dyn, (int)Exec::bwd_smem_bytes(16, bwd_ld(8))));
  CUDA_TRY(cudaFuncSetAttribute(bwd_step_kernel<4, 16>, dyn, (int)Exec::bwd_smem_bytes(32, bwd_ld(16))));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<1, 8, 2>, dyn, (int)bwd_stream_smem_bytes<1, 8, 2>()));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<2, 8, 2>, dyn, (int)bwd_stream_smem_bytes<2, 8, 2>()));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<4, 16, 2>, dyn, (int)bwd_stream_smem_bytes<4, 16, 2>()));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<1, 8, 1>, dyn, (int)bwd_stream_smem_bytes<1, 8, 1>()));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<2, 8, 1>, dyn, (int)bwd_stream_smem_bytes<2, 8, 1>()));
  CUDA_TRY(cudaFuncSetAttribute(bwd_stream_kernel<4, 16, 1>, dyn, (int)bwd_stream_smem_bytes<4, 16, 1>()));
  CUDA_TRY(cudaFuncSetAttribute(dw_slab_kernel<false>, dyn, (int)dws_smem_bytes<false>()));
  CUDA_TRY(cudaFuncSetAttribute(dw_slab_kernel<true>, dyn, (int)dws_smem_bytes<true>()));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<1, false>, dyn, (int)dw_smem_bytes<1, false>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<2, false>, dyn, (int)dw_smem_bytes<2, false>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<4, false>, dyn, (int)dw_smem_bytes<4, false>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<8, false>, dyn, (int)dw_smem_bytes<8, false>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<1, true>, dyn, (int)dw_smem_bytes<1, true>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<2, true>, dyn, (int)dw_smem_bytes<2, true>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<4, true>, dyn, (int)dw_smem_bytes<4, true>(DW_WINDOW)));
  CUDA_TRY(cudaFuncSetAttribute(dw_kernel<8, true>, dyn, (int)dw_smem_bytes<8, true>(DW_WINDOW)));
  g_smem_opted_in[dev] = true;
  return SNN_OK;
}
}  // namespace

extern "C" snn_status snn_train_step(snn_net* net, const snn_step_args* a, float* loss_host_out) {
  if (!net) return SNN_ERR_INVALID_ARG;
  if (!a || !loss_host_out) return fail(net, SNN_ERR_INVALID_ARG, "null argument");
  const int L = net->L, T = a->T, B = a->B;
  const bool fwd_only = (a->flags & SNN_FLAG_FORWARD_ONLY) != 0;
  if (T < 1 || B < 1) return fail(net, SNN_ERR_INVALID_ARG, "T and B must be >= 1");
  if (B > 65535) return fail(net, SNN_ERR_UNSUPPORTED, "batch above 65535");
  if (!a->input || !a->targets || !a->W_ff || !a->W_rec || !a->W_out || !a->device_ws)
    return fail(net, SNN_ERR_INVALID_ARG, "null pointer in arguments");
  if (!fwd_only && (!a->dW_ff || !a->dW_rec || !a->dW_out))
    return fail(net, SNN_ERR_INVALID_ARG, "null gradient pointer");
  for (int l = 0; l < L; ++l) {
    if (!a->W_ff[l] || !a->W_rec[l]) return fail(net, SNN_ERR_INVALID_ARG, "null weight pointer");
    if (!fwd_only && (!a->dW_ff[l] || !a->dW_rec[l])) return fail(net, SNN_ERR_INVALID_ARG, "null gradient pointer");
    if ((reinterpret_cast<uintptr_t>(a->W_ff[l]) | reinterpret_cast<uintptr_t>(a->W_rec[l])) % 16 != 0)
      return fail(net, SNN_ERR_INVALID_ARG, "weights must be 16-byte aligned");
    if (!fwd_only &&
        (reinterpret_cast<uintptr_t>(a->dW_ff[l]) | reinterpret_cast<uintptr_t>(a->dW_rec[l])) % 16 != 0)
      return fail(net, SNN_ERR_INVALID_ARG, "gradients must be 16-byte aligned");
  }
  if (net->cell == SNN_CELL_LIF && a->input_format != SNN_INPUT_BITS)
    return fail(net, SNN_ERR_UNSUPPORTED, "the LIF cell takes bit-packed input (SNN_INPUT_BITS)");
  if (net->cell == SNN_CELL_GRADED && a->input_format != SNN_INPUT_DENSE)
    return fail(net, SNN_ERR_UNSUPPORTED, "the graded cell takes dense fp32 input (SNN_INPUT_DENSE)");
  if (!(a->max_activity > 0.f) || a->max_activity > 1.f) return fail(net, SNN_ERR_INVALID_ARG, "max_activity not in (0, 1]");
  if ((a->flags & SNN_FLAG_BACKWARD_EVENT_DRIVEN) && (net->surrogate != SNN_SURR_TRIANGLE || net->cell != SNN_CELL_LIF))
    return fail(net, SNN_ERR_UNSUPPORTED, "the event-driven backward pass needs SNN_SURR_TRIANGLE and the LIF cell");
  if (reinterpret_cast<uintptr_t>(a->device_ws) % ALIGN != 0)
    return fail(net, SNN_ERR_INVALID_ARG, "device workspace must be 256-byte aligned");

  Exec ex;
  ex.net = net; ex.a = a; ex.L = L; ex.B = B; ex.T = T;
  std::string why;
  if (!compute_layout(net, T, B, &a->ckpt, a->max_activity, a->flags, ex.lo, why))
    return fail(net, SNN_ERR_INVALID_ARG, "%s", why.c_str());
  const Layout& lo = ex.lo;
  const size_t pinned_states = lo.tier2_on_device ? 0 : (size_t)lo.n_remote * lo.state_bytes;
  const size_t pinned_need = pinned_states + (lo.spill ? (size_t)lo.ev_segments * lo.ev_window_bytes : 0);
  if (a->device_ws_bytes < lo.total)
    return fail(net, SNN_ERR_WORKSPACE_TOO_SMALL, "device workspace %zu < %zu bytes", a->device_ws_bytes, lo.total);
  if (pinned_need > 0 && (!a->pinned_ws || a->pinned_ws_bytes < pinned_need))
    return fail(net, SNN_ERR_WORKSPACE_TOO_SMALL, "pinned workspace %zu < %zu bytes", a->pinned_ws_bytes, pinned_need);
  std::vector<snn_op> ops;
  {
    int n_ops = 0;
    snn_plan(T, &a->ckpt, nullptr, 0, &n_ops, nullptr, nullptr);
    ops.resize(n_ops);
    snn_plan(T, &a->ckpt, ops.data(), n_ops, &n_ops, nullptr, nullptr);
  }
  ex.ws = static_cast<char*>(a->device_ws);
  ex.main = (cudaStream_t)a->main_stream;
  ex.side = a->side_stream ? (cudaStream_t)a->side_stream : ex.main;
  ex.remote_tier = lo.n_remote > 0;
  ex.slot_event.assign(lo.n_local, -1);
  ex.timed = (a->flags & SNN_FLAG_TIME_PHASES) != 0;
  if (!net->ev_main) {
    CUDA_TRY(cudaEventCreateWithFlags(&net->ev_main, cudaEventDisableTiming));
  }
  {
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (const snn_status os = opt_in_shared_memory(net, dev); os != SNN_OK) return os;
    if (net->device != dev) {   // figures cached per net belong to the device they were asked of
      net->device = dev;
      net->coop_sms = -1;
      net->fwd_segment_capacity[0] = net->fwd_segment_capacity[1] = -1;
      for (int& c : net->bwd_stream_capacity) c = -1;
    }
  }
  cudaStream_t ms = ex.main;
  const auto& sz = net->sizes;

  // Everything the step enqueues; an error ends the enqueueing, and the caller below still waits for both
  // streams before it returns, so no work is in flight on the caller's buffers after any return.
  NvtxRange step_range("snn_train_step");
  auto enqueue = [&]() -> snn_status {
  // ---- start-of-step state: status, counts, delta carry, list offsets, spikes at t = 0, gradients
  CUDA_TRY(cudaMemsetAsync(ex.ws + lo.status, 0, 256, ms));
  CUDA_TRY(cudaMemsetAsync(ex.ws + lo.counts, 0, 4 * (size_t)B * sz[L], ms));
  CUDA_TRY(cudaMemsetAsync(ex.ws + lo.carry[0], 0, lo.state_bytes, ms));
  CUDA_TRY(cudaMemsetAsync(ex.ws + lo.carry[1], 0, lo.state_bytes, ms));
  for (int l = 0; l <= L; ++l) {
    CUDA_TRY(cudaMemsetAsync(ex.ws + lo.off[l], 0, 4 * (size_t)2 * B, ms));
    if (l > 0) CUDA_TRY(cudaMemsetAsync(ex.ws + lo.mask[l], 0, 4 * (size_t)B * lo.words[l], ms));
  }
  if (!fwd_only) {
    for (int l = 1; l <= L; ++l) {
      CUDA_TRY(cudaMemsetAsync(a->dW_ff[l - 1], 0, 4 * (size_t)sz[l - 1] * sz[l], ms));
      CUDA_TRY(cudaMemsetAsync(a->dW_rec[l - 1], 0, 4 * (size_t)sz[l] * sz[l], ms));
    }
  }
  if (a->flags & SNN_FLAG_INPUT_ON_HOST) {
    CUDA_TRY(cudaMemcpyAsync(ex.ws + lo.in_stage, a->input,
                             4 * (size_t)T * B * (net->cell == SNN_CELL_GRADED ? sz[0] : lo.words[0]),
                             cudaMemcpyHostToDevice, ms));
    CUDA_TRY(cudaMemcpyAsync(ex.ws + lo.tg_stage, a->targets, 4 * (size_t)B, cudaMemcpyHostToDevice, ms));
  }

  if (net->cell == SNN_CELL_GRADED) {   // spike words of the dense input, all steps at once
    const size_t n_rows = (size_t)T * B, n_warps = n_rows * lo.words[0];
    dense_to_words_kernel<<<(unsigned)((n_warps * 32 + 255) / 256), 256, 0, ms>>>(
        reinterpret_cast<const float*>(ex.in_base()), n_rows, sz[0], lo.words[0], ex.at<uint32_t>(lo.in_words));
    ++ex.launches;
    CUDA_TRY(cudaGetLastError());
  }
  int last_fwd = -1;
  for (int i = 0; i < (int)ops.size(); ++i)
    if (ops[i].kind == SNN_OP_FWD) last_fwd = i;
  snn_status st = SNN_OK;
  static const char* const op_names[] = {"snn:forward", "snn:re-forward 1", "snn:re-forward 2", "snn:backward",
                                         "snn:checkpoint to host", "snn:checkpoint from host", "snn:clear state"};
  for (int i = 0; i < (int)ops.size() && st == SNN_OK; ++i) {
    const snn_op& op = ops[i];
    NvtxRange range(op.kind >= 0 && op.kind <= SNN_OP_ZERO ? op_names[op.kind] : "snn:op");
    switch (op.kind) {
      case SNN_OP_ZERO:
        st = ex.wait_slot(op.keep_slot);
        if (st == SNN_OK)
          CUDA_TRY(cudaMemsetAsync(ex.ws + lo.slots + (size_t)op.keep_slot * lo.state_bytes, 0, lo.state_bytes, ms));
        break;
      case SNN_OP_FWD: {
        const int seg = op.t0 / lo.ev_steps;
        if (lo.spill && seg != ex.ev_seg) st = ex.ev_enter_forward(seg);
        if (st == SNN_OK) st = ex.run_forward(op, true);
        if (st == SNN_OK && (i == last_fwd || lo.spill)) st = ex.run_flush(op.t1);
        if (st == SNN_OK && lo.spill && i != last_fwd) st = ex.ev_copy(seg & 1, seg, true);   // behind the forward pass
        if (st == SNN_OK && i == last_fwd) st = ex.run_readout();
        break;
      }
      case SNN_OP_REFWD1:
      case SNN_OP_REFWD2:
      case SNN_OP_BWD: {
        const int seg = op.t0 / lo.ev_steps;
        if (lo.spill && seg != ex.ev_seg) st = ex.ev_enter_backward(seg);
        if (st == SNN_OK) st = op.kind == SNN_OP_BWD ? ex.run_backward(op) : ex.run_forward(op, false);
        break;
      }
      case SNN_OP_D2H:
      case SNN_OP_H2D:
        st = ex.run_copy(op);
        break;
      default:
        st = fail(net, SNN_ERR_INVALID_ARG, "unknown op");
    }
    if (fwd_only && i == last_fwd) break;
  }
  return st;
  };
  const snn_status st = enqueue();
  // ---- finish: everything on both streams, then status and loss
  cudaError_t e1 = cudaStreamSynchronize(ex.side);
  cudaError_t e2 = cudaStreamSynchronize(ex.main);
  if (st != SNN_OK) return st;
  if (e1 != cudaSuccess || e2 != cudaSuccess)
    return fail(net, SNN_ERR_CUDA, "stream synchronize failed: %s", cudaGetErrorString(e1 != cudaSuccess ? e1 : e2));
  uint32_t host_status[2] = {0, 0};
  CUDA_TRY(cudaMemcpy(host_status, ex.ws + lo.status, 8, cudaMemcpyDeviceToHost));
  std::memcpy(loss_host_out, &host_status[1], 4);

  if (a->flags & SNN_FLAG_TIME_PHASES) ex.collect_spans();
  net->dev_peak = lo.total;
  net->pin_peak = pinned_need;
  (void)pinned_states;
  net->stats.state_bytes = lo.state_bytes;
  net->stats.local_state_slots = lo.n_local;
  net->stats.remote_state_slots = lo.n_remote;
  net->stats.d2h_copies = ex.d2h;
  net->stats.h2d_copies = ex.h2d;
  net->stats.kernel_launches = ex.launches;
  net->stats.event_bytes = lo.event_bytes;
  net->stats.event_window_copies = ex.ev_copies;
  net->ev_layout.assign(lo.spill ? 0 : L + 1, snn_event_layout{});   // spilled events are not all on the device
  for (int l = 0; l <= L && !lo.spill; ++l) {
    snn_event_layout& e = net->ev_layout[l];
    e.offsets_off = lo.off[l]; e.pool_off = lo.pool[l]; e.values_off = lo.vals[l]; e.pool_capacity = lo.cap[l];
    e.mask_off = lo.mask[l]; e.mask_words = lo.words[l];
  }
  if ((host_status[0] & STATUS_DEBUG_CHECK) || ex.debug_violation)
    return fail(net, SNN_ERR_DEBUG_CHECK, "an index check of the bounds-checked build failed (%s)",
                ex.debug_violation ? "state slot outside the layout" : "event position or row index out of range");
  if (host_status[0] & STATUS_BAD_TARGET)
    return fail(net, SNN_ERR_INVALID_ARG, "a target is outside [0, %d)", sz[L + 1]);
  if (host_status[0] & STATUS_SYNC_TIMEOUT)
    return fail(net, SNN_ERR_DEVICE_TIMEOUT, "a thread block gave up waiting for the spikes of another one");
  if (host_status[0] & STATUS_EVENT_OVERFLOW)
    return fail(net, SNN_ERR_EVENT_OVERFLOW, "more events than max_activity=%g allows", (double)a->max_activity);
  return SNN_OK;
}

// Self-test of the bounded waits between thread blocks (see snn.h).
extern "C" snn_status snn_selftest_wait_timeout(void* device_scratch, uint32_t poll_limit, void* stream) {
  if (!device_scratch || poll_limit == 0) return SNN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t* words = reinterpret_cast<uint32_t*>(device_scratch);
  if (cudaMemsetAsync(words, 0, 256, st) != cudaSuccess) return SNN_ERR_CUDA;
  wait_selftest_kernel<<<1, 64, 0, st>>>(words, words + 32, poll_limit);
  uint32_t host[2] = {0, 0};
  if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess ||
      cudaMemcpy(host, words, 8, cudaMemcpyDeviceToHost) != cudaSuccess)
    return SNN_ERR_CUDA;
  return (host[0] & STATUS_SYNC_TIMEOUT) && host[1] == 0 ? SNN_ERR_DEVICE_TIMEOUT : SNN_OK;
}

// ------------------------------------------------------------------------------------------
// Training step on the library's own, statically reserved device workspace, for callers that
// have no way to allocate device memory when the step is due (no PyTorch in the process, the
// whole device already given to another pool, or a fixed budget under which cudaMalloc could
// fail or stall the device).  The buffer lives in the device image of this library: every GPU
// that loads it holds SNN_STATIC_WORKSPACE_BYTES until exit.
//
// The array's name is only a handle in host code; the device address that kernels and copies
// need comes from cudaGetSymbolAddress, looked up once per device with that device current.
static __device__ __align__(256) unsigned char g_static_workspace[SNN_STATIC_WORKSPACE_BYTES];

namespace {
void* g_static_workspace_addr[kMaxDevices] = {nullptr};   // guarded by g_device_mutex
}  // namespace

extern "C" snn_status snn_train_step_static(snn_net* net, const snn_step_args* args, float* loss_host_out) {
  if (!net) return SNN_ERR_INVALID_ARG;
  if (!args || !loss_host_out) return fail(net, SNN_ERR_INVALID_ARG, "null argument");
  if (args->T < 1 || args->B < 1) return fail(net, SNN_ERR_INVALID_ARG, "T and B must be >= 1");
  if (!(args->max_activity > 0.f) || args->max_activity > 1.f)
    return fail(net, SNN_ERR_INVALID_ARG, "max_activity not in (0, 1]");
  // size check first: nothing runs for a step that does not fit the built-in buffer
  Layout lo;
  std::string why;
  if (!compute_layout(net, args->T, args->B, &args->ckpt, args->max_activity, args->flags, lo, why))
    return fail(net, SNN_ERR_INVALID_ARG, "%s", why.c_str());
  if (lo.total > (size_t)SNN_STATIC_WORKSPACE_BYTES)
    return fail(net, SNN_ERR_WORKSPACE_TOO_SMALL,
                "this step needs %zu bytes of device workspace; the built-in workspace holds %zu "
                "(use snn_train_step with a caller-provided workspace)",
                lo.total, (size_t)SNN_STATIC_WORKSPACE_BYTES);
  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(net, SNN_ERR_UNSUPPORTED, "device index %d out of range", dev);
  void* ws_addr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_device_mutex);
    if (!g_static_workspace_addr[dev]) {  // first call on this device: resolve the buffer's device address
      void* p = nullptr;
      CUDA_TRY(cudaGetSymbolAddress(&p, g_static_workspace));
      if (!p) return fail(net, SNN_ERR_CUDA, "built-in workspace has no device address");
      g_static_workspace_addr[dev] = p;
    }
    ws_addr = g_static_workspace_addr[dev];
  }
  snn_step_args a = *args;
  a.device_ws = ws_addr;
  a.device_ws_bytes = (size_t)SNN_STATIC_WORKSPACE_BYTES;
  return snn_train_step(net, &a, loss_host_out);
}
