/*
 * snn.h — C ABI of the BPTT training step for sparse recurrent / spiking networks
 * under the gradient-checkpointing strategies of "Optimal Gradient Checkpointing
 * for Sparse and Recurrent Architectures using Off-Chip Memory" (arXiv 2412.11810).
 *
 * Strategy names follow the caption of the paper's Fig. 1:
 *   STANDARD  every membrane state of every step kept ("Base Implementation", Eq. 2)
 *   CHUNK     local checkpoints every chunk_size steps, one recomputation pass
 *             (section "Standard Checkpointing", Eqs. 1, 4, 5)
 *   REMOTE    the same schedule with the checkpoints in remote memory (Eqs. 6, 7)
 *   DOUBLE    remote checkpoints every remote_chunk_size steps, local ones every
 *             chunk_size steps recomputed by an extra pass (Eqs. 11-13)
 *   HIERARCHICAL  checkpoints every chunk_size steps kept in remote memory and moved nb_local at a
 *             time, the last nb_local staying local (section "Hierarchical Checkpointing", Eqs. 8-10)
 *   DOUBLE_LOCAL  the schedule of DOUBLE with both tiers in device memory (Discussion: the purely
 *             on-chip use of Double Checkpointing)
 * "Local" memory is device memory, "remote" memory is pinned host memory.
 *
 * General rules.  Every function returns an snn_status and never throws, aborts
 * or exits.  The library allocates no device or pinned memory: the caller passes
 * two workspaces sized by snn_workspace_query and the library carves them up.
 * Pointers marked "device" must be device pointers on the current CUDA device;
 * pointers marked "host" are ordinary host pointers; "pinned" means page-locked
 * host memory.  All floating-point data is fp32, all matrices row-major with the
 * presynaptic neuron as the row: W_ff^l [N_{l-1}][N_l], W_rec^l [N_l][N_l],
 * W_out [N_L][N_out].
 */
#ifndef SNN_H_
#define SNN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct snn_net snn_net; /* opaque; host-side descriptors only */

typedef enum {
  SNN_OK = 0,
  SNN_ERR_INVALID_ARG = 1,
  SNN_ERR_WORKSPACE_TOO_SMALL = 2,
  SNN_ERR_EVENT_OVERFLOW = 3, /* more events than max_activity allows; gradients unspecified */
  SNN_ERR_DEVICE_TIMEOUT = 4,
  SNN_ERR_CUDA = 5,
  SNN_ERR_UNSUPPORTED = 6,
  SNN_ERR_DEBUG_CHECK = 7 /* bounds-checked build only: an index check failed; nothing was accessed out of bounds */
} snn_status;

typedef enum { SNN_STANDARD = 0, SNN_CHUNK = 1, SNN_REMOTE = 2, SNN_DOUBLE = 3, SNN_HIERARCHICAL = 4,
               SNN_DOUBLE_LOCAL = 5 } snn_strategy;
typedef enum { SNN_CELL_LIF = 0, SNN_CELL_GRADED = 1 } snn_cell;
/* Pseudo-derivative of the spike, x = V - threshold.  The paper names none; 0 is the default of the
 * benchmark definition.  0: 1 / (1 + beta |x|)^2.  1: beta s (1 - s), s = sigmoid(beta x).
 * 2 (an extension): beta max(0, 1 - beta |x|), zero outside |x| < 1 / beta. */
typedef enum { SNN_SURR_FAST_SIGMOID = 0, SNN_SURR_SIGMOID = 1, SNN_SURR_TRIANGLE = 2 } snn_surrogate;

#define SNN_MAX_LAYERS 8      /* hidden layers                                   */
#define SNN_MAX_NEURONS 65536 /* per layer; hidden sizes must be multiples of 4  */

/* Network description.  The paper trains "by BPTT using the surrogate gradient
 * approach" (Methods, "BPTT based SNN training") and prints no neuron equations;
 * this library fixes them as
 *   I      = S^{l-1}_t W_ff^l + S^l_{t-1} W_rec^l      (one accumulator per neuron,
 *            feed-forward events first, then recurrent, ascending presynaptic index)
 *   V^l_t  = fma(alpha, V^l_{t-1}, I) - theta S^l_{t-1}    LIF, alpha = exp(-1/tau_mem)
 *   S^l_t  = [V^l_t > theta]
 *   graded cell: no reset, S^l_t = V^l_t [V^l_t > theta]
 *   loss   = mean soft-max cross-entropy of readout_scale * (sum_t S^L_t) W_out
 *   backward: delta_t = g_S sigma'(V_t - theta) + alpha delta_{t+1} with
 *             sigma'(x) = 1/(1+beta|x|)^2 (fast sigmoid) or beta s(beta x)(1-s(beta x)). */
typedef struct {
  int32_t n_sizes;      /* L + 2                                               */
  const int32_t* sizes; /* host: N_0, N_1 .. N_L, N_out (copied)               */
  float tau_mem;        /* membrane time constant in steps, > 0                */
  float threshold;      /* theta                                               */
  int32_t surrogate;    /* snn_surrogate                                       */
  float surrogate_beta; /* beta > 0                                            */
  int32_t cell;         /* snn_cell                                            */
  float readout_scale;  /* multiplies the time-summed readout                  */
} snn_config;

/* Validates the description and creates the host-side object.  No device work.
 * Errors: SNN_ERR_INVALID_ARG (null, sizes < 1, tau/beta <= 0),
 * SNN_ERR_UNSUPPORTED (more than SNN_MAX_LAYERS hidden layers, a hidden size that
 * is not a multiple of 4 or exceeds SNN_MAX_NEURONS). */
snn_status snn_create(const snn_config* cfg, snn_net** out);
void snn_destroy(snn_net* net);

/* The leak alpha = exp(-1/tau_mem), evaluated in double and rounded once to fp32. */
float snn_alpha(const snn_net* net);

/* 1 if the library was compiled with -DSNN_DEBUG_CHECKS=1 (libsnnckpt_debug.so), else 0.  That build tests the
 * data-dependent indices of the gather kernels (position in an event pool, presynaptic row of an event) and the state
 * slots the executor addresses before use; a bad index is replaced by a valid one and the step returns
 * SNN_ERR_DEBUG_CHECK.  Results of a correct step are bit-identical to the ordinary build. */
int32_t snn_debug_checks_enabled(void);

/* Checkpoint hyper-parameters (paper: chunk_size, Eq. 1; remote_chunk_size, Eq. 11; nb_local, Eq. 8).
 * STANDARD ignores all; CHUNK and REMOTE need chunk_size >= 1; DOUBLE and DOUBLE_LOCAL need
 * remote_chunk_size >= chunk_size >= 1 and remote_chunk_size % chunk_size == 0; HIERARCHICAL needs
 * chunk_size >= 1 and nb_local >= 1.
 * The sequence length need not be a multiple of any of them: the last segment is short. */
typedef struct {
  int32_t strategy; /* snn_strategy */
  int32_t chunk_size;
  int32_t remote_chunk_size;
  int32_t nb_local;
} snn_ckpt;

/* Hyper-parameters by the rules of the paper's Hyperparameter Study: CHUNK chunk_size = sqrt(T);
 * DOUBLE remote_chunk_size within 64 .. 256 (256 once T >= 1024, else the power of two nearest T/4,
 * at least 4) and chunk_size = sqrt(remote_chunk_size); REMOTE the largest chunk_size whose device
 * workspace fits device_budget_bytes (sqrt(T) if the budget is 0); HIERARCHICAL chunk_size =
 * sqrt(T) and nb_local = sqrt(number of checkpoints).  Host only.  net, B and max_activity are
 * used for the REMOTE rule only (net may be NULL otherwise). */
snn_status snn_suggest_ckpt(const snn_net* net, int32_t T, int32_t B, int32_t strategy, size_t device_budget_bytes,
                            float max_activity, snn_ckpt* out);

/* Bytes of device and pinned-host workspace a train step of T steps and batch B needs.
 * max_activity in (0, 1]: upper bound on the mean fraction of active neurons per layer
 * over the sequence; it sizes the per-sample event pools (the sparse activations of the
 * whole sequence stay in device memory, as in the paper's Discussion). */
snn_status snn_workspace_query(const snn_net* net, int32_t T, int32_t B, const snn_ckpt* ckpt,
                               float max_activity, size_t* device_bytes, size_t* pinned_bytes);

/* The same for a step that will run with the given SNN_FLAG_* bits: SNN_FLAG_INPUT_ON_HOST adds a staging
 * area for the input and the targets (T B N_0 values resp. T B ceil(N_0/32) words); snn_workspace_query
 * is this call with flags = 0.  snn_train_step checks the workspace against the flags it is given. */
snn_status snn_workspace_query_flags(const snn_net* net, int32_t T, int32_t B, const snn_ckpt* ckpt,
                                     float max_activity, uint32_t flags, size_t* device_bytes,
                                     size_t* pinned_bytes);

#define SNN_INPUT_BITS 0  /* uint32 [T][B][ceil(N_0/32)], bit i%32 of word i/32 = spike of input i; bits at
                             positions >= N_0 of a row's last word are ignored                          */
#define SNN_INPUT_DENSE 1 /* fp32 [T][B][N_0], zero = no event (graded cell)                        */

#define SNN_FLAG_INPUT_ON_HOST 1u /* input and targets are pinned host pointers; copied in the call */
#define SNN_FLAG_FORWARD_ONLY 2u  /* forward pass, readout and loss only                            */
#define SNN_FLAG_TIME_PHASES 4u   /* bracket every pass with CUDA events (see snn_phase_times_get)  */
/* The backward pass has two launch orders.  Wavefront: one launch per step covers all layers and also
 * multiplies by W_ff of the layer above.  Layer by layer: runs of 32 steps, the feed-forward term of a
 * whole run computed as one product so that W_ff is streamed once per run.  By default the second is
 * used unless the network is small enough for the backward pass of a segment to run as one launch with the
 * weights in shared memory (see SNN_FLAG_BACKWARD_PER_STEP); these flags force one or the other.
 * Gradients are bit-identical across strategies for a given order, not between the two orders. */
#define SNN_FLAG_BACKWARD_LAYER_BY_LAYER 8u
#define SNN_FLAG_BACKWARD_WAVEFRONT 16u
/* The recomputation passes take two launches per run of steps (the input currents of all its steps from the
 * stored events at once, thread blocks ordered so that those that run together gather from the same columns;
 * then the leak/reset recurrence); this flag forces one launch per step.  Results are bit-identical either way. */
#define SNN_FLAG_REFORWARD_PER_STEP 32u
/* Networks whose weights exceed L2 compute those input currents with the weight rows as the stationary
 * operand instead: a thread block reads each row of its column slab once per run and adds it to every
 * (step, sample) of the run in which that neuron fired (spiking cell).  This flag forces that order for
 * smaller networks, and for the graded cell (each event then multiplies the row by its value), too.  Results are
 * bit-identical either way. */
#define SNN_FLAG_REFORWARD_ROWS 512u
/* The forward pass of a spiking (LIF) network whose weights fit in L2 runs as one cooperative launch per
 * forward operation of the plan when the device can hold all its thread blocks at once: blocks wait for
 * each other's spike words sample by sample instead of once per launch.  This flag forces one launch per
 * step.  Results are bit-identical either way.  A wait that does not end within a few seconds makes the
 * step return SNN_ERR_DEVICE_TIMEOUT. */
#define SNN_FLAG_FORWARD_PER_STEP 64u
/* Small spiking networks (batch up to 64; the columns of W_ff and W_rec that 16 neurons need within
 * 200 KB; at most one thread block of 16 neurons per SM over all layers) keep their weights in shared
 * memory during a forward launch.  This flag makes them stream the weights from L2 like larger ones. */
#define SNN_FLAG_FORWARD_STREAM_WEIGHTS 128u
/* Networks small enough that 32 rows of a layer's recurrent and next feed-forward matrix fit in shared
 * memory beside the staging buffers (per cluster rank) run the backward pass of a segment as one
 * cooperative launch with those weights resident.  This flag forces one launch per step.  Results are
 * bit-identical either way. */
#define SNN_FLAG_BACKWARD_PER_STEP 256u
/* The feed-forward product of the layer-by-layer order runs on the tcgen05 tensor cores (accumulator in tensor
 * memory).  This flag selects the older mma.sync kernel instead; the two agree to rounding (both are three-pass
 * tf32 products with fp32 accumulation), not bit for bit. */
#define SNN_FLAG_FF_PRODUCT_MMA_SYNC 1024u
/* The paper keeps the sparse activations of the whole sequence in local memory (Discussion).  With this flag
 * (REMOTE and DOUBLE only; ignored otherwise) the device holds the events of two remote segments at a time (chunk_size
 * steps for REMOTE, remote_chunk_size for DOUBLE): each segment's events are copied to the pinned workspace on the side
 * stream behind the forward pass and fetched one segment ahead of the backward pass, ordered with events like the
 * state checkpoints.  max_activity then bounds the mean activity per segment.  snn_workspace_query_flags reports the
 * sizes; snn_get_event_layout is not available for such a step.  Gradients are bit-identical to the unspilled step. */
#define SNN_FLAG_SPILL_EVENTS 2048u
/* Event-driven backward pass (an extension in the spirit of the paper's Discussion: exploit the sparse activations).
 * With SNN_SURR_TRIANGLE the pseudo-derivative is zero unless |V - threshold| < 1 / beta, so only the rows of W_rec and
 * W_ff of near-threshold (sample, neuron) pairs are read and multiplied; everywhere else delta_t = alpha delta_{t+1}.
 * Pays when batch x fraction of near-threshold neurons is well below one; otherwise the dense tensor-core kernels,
 * which read every row once for the whole batch, are faster.  SNN_ERR_UNSUPPORTED for other surrogates or the graded
 * cell.  Gradients are bit-identical across strategies under this flag, and agree with the dense orders to rounding. */
#define SNN_FLAG_BACKWARD_EVENT_DRIVEN 4096u
/* The weight gradient of a segment (the sparse outer product of Methods, "BPTT based SNN training") has two kernels.
 * One gathers, per presynaptic row, the delta rows of the (step, sample) pairs in which it fired; the other keeps a slab
 * of the deltas in shared memory and streams the rows of dW past it, so that dW is read and written once per 128 pairs
 * and nothing is gathered from L2 (the default when the weights exceed 96 MB).  These flags force one or the other.
 * Results are bit-identical either way. */
#define SNN_FLAG_WEIGHT_GRADIENT_GATHER 8192u
#define SNN_FLAG_WEIGHT_GRADIENT_SLAB 16384u

typedef struct {
  int32_t T, B;
  const void* input;      /* device (or pinned host with SNN_FLAG_INPUT_ON_HOST), read-only       */
  int32_t input_format;   /* SNN_INPUT_BITS | SNN_INPUT_DENSE                                      */
  const int32_t* targets; /* [B], same memory space as input; each in [0, N_out), else the step
                             returns SNN_ERR_INVALID_ARG (checked on the device, never used as an index) */
  const float* const* W_ff;  /* host array of L device pointers                                   */
  const float* const* W_rec; /* host array of L device pointers                                   */
  const float* W_out;        /* device                                                            */
  float* const* dW_ff;       /* host array of L device pointers; OVERWRITTEN with the gradient    */
  float* const* dW_rec;      /* of the mean loss                                                  */
  float* dW_out;
  void* device_ws;  size_t device_ws_bytes; /* device, 256-byte aligned                           */
  void* pinned_ws;  size_t pinned_ws_bytes; /* pinned host; may be NULL for STANDARD and CHUNK    */
  void* main_stream; /* cudaStream_t for the kernels                                              */
  void* side_stream; /* cudaStream_t for checkpoint copies; must differ from main_stream for
                        REMOTE and DOUBLE if copies are to overlap recomputation                  */
  snn_ckpt ckpt;
  float max_activity;
  uint32_t flags;
  float* const* debug_V; /* optional host array of L device pointers [T+1][B][N_l]: the forward
                            pass also stores every membrane state there (index 0 untouched)       */
} snn_step_args;

/* One BPTT training step (paper, Fig. 1: forward, recomputation passes, backward) for the
 * given strategy.  Returns the loss through loss_host_out (host) and the gradients in the
 * dW buffers; synchronous: all work on both streams has finished on return.  Gradients of
 * every checkpointing strategy are bit-identical to those of SNN_STANDARD.
 * Errors: SNN_ERR_INVALID_ARG (nulls, T < 1, B < 1, bad intervals, misaligned workspace),
 * SNN_ERR_WORKSPACE_TOO_SMALL, SNN_ERR_UNSUPPORTED (input format / cell mismatch) — all
 * before any kernel is launched; SNN_ERR_EVENT_OVERFLOW, SNN_ERR_CUDA after. */
snn_status snn_train_step(snn_net* net, const snn_step_args* args, float* loss_host_out);

/* The same training step for callers that cannot allocate device memory at all.
 * (The paper has no counterpart: this entry point exists for embedding only.)
 * Some hosts of this library own no allocator they may call when a step is due: a C program
 * that links the library without PyTorch, a process whose device memory has been handed over
 * entirely to another component's pool, or a service under a fixed memory budget where a
 * cudaMalloc at step time could fail, or would stall every stream of the device while it runs.
 * For them the device workspace is not passed in: the library uses a buffer of
 * SNN_STATIC_WORKSPACE_BYTES that is part of its own device image.  Every GPU that loads the
 * library holds those bytes until the process exits, whether this entry point is used or not.
 *   - args->device_ws and args->device_ws_bytes are ignored; inputs, targets, weights, gradient
 *     buffers, the pinned workspace (REMOTE / DOUBLE) and the streams are passed as usual.
 *   - A step whose snn_workspace_query device size exceeds SNN_STATIC_WORKSPACE_BYTES is
 *     rejected with SNN_ERR_WORKSPACE_TOO_SMALL before anything runs.
 *   - The call allocates and frees no device or pinned memory.  The first call on a device looks
 *     up the address of the built-in buffer (once per device, with that device current); make
 *     that first call outside any stream capture.  Like snn_train_step it creates a few CUDA
 *     events the first time a net is used.
 *   - All calls on one device share the one buffer.  It keeps whatever the previous call left;
 *     the step clears everything it needs to start from zero.  Two calls that overlap on the GPU
 *     (different host threads, different nets, different streams) race on it: serialise them.
 * Results are those of snn_train_step, bit for bit. */
#define SNN_STATIC_WORKSPACE_BYTES (32u << 20)
snn_status snn_train_step_static(snn_net* net, const snn_step_args* args, float* loss_host_out);

/* High-water marks of the last train step: bytes of the device workspace and of the pinned
 * workspace actually used, and the part of the former that scales with the paper's M_s
 * (number of dense states held locally times bytes per state; Eqs. 2, 4, 6, 11). */
snn_status snn_peak_memory(const snn_net* net, size_t* device_peak_bytes, size_t* pinned_peak_bytes);
typedef struct {
  size_t state_bytes;         /* M_s = 4 B sum_l N_l                              */
  int32_t local_state_slots;  /* dense states held in device memory               */
  int32_t remote_state_slots; /* dense states held in pinned memory               */
  int32_t d2h_copies, h2d_copies; /* checkpoint transfers of the last step        */
  int32_t kernel_launches;    /* kernels launched by the last step                */
  size_t event_bytes;         /* event pools + spike masks held on the device (scale with T, or with the
                                 remote segment under SNN_FLAG_SPILL_EVENTS)      */
  int32_t event_window_copies; /* event-window transfers of the last step (SNN_FLAG_SPILL_EVENTS) */
} snn_memory_stats;
snn_status snn_memory_stats_get(const snn_net* net, snn_memory_stats* out);

/* Device time of the last step per pass of Fig. 1, measured with CUDA events on the main stream
 * when the step ran with SNN_FLAG_TIME_PHASES, and the kernels launched in each.  BWD is the
 * surrogate-gradient step kernel, DW the sparse outer-product weight-gradient kernel; D2H and H2D are the
 * checkpoint copies, timed on the side stream (their `launches` count copies; they overlap the passes);
 * FFGEMM is the time-batched feed-forward product of the layer-by-layer backward order. */
typedef enum { SNN_PHASE_FWD = 0, SNN_PHASE_REFWD1 = 1, SNN_PHASE_REFWD2 = 2, SNN_PHASE_BWD = 3,
               SNN_PHASE_DW = 4, SNN_PHASE_READOUT = 5, SNN_PHASE_D2H = 6, SNN_PHASE_H2D = 7,
               SNN_PHASE_FFGEMM = 8, SNN_N_PHASES = 9 } snn_phase;
typedef struct {
  float ms[SNN_N_PHASES];
  int32_t launches[SNN_N_PHASES];
} snn_phase_times;
snn_status snn_phase_times_get(const snn_net* net, snn_phase_times* out);

const char* snn_last_error(const snn_net* net); /* owned by net; valid until the next call */

/* ---- schedule (host only) --------------------------------------------------------------
 * The execution trace of Fig. 1 as a list of segment operations over numbered state slots.
 * FWD / REFWD1 / REFWD2 compute V_{t0+1} .. V_{t1} from V_{t0} held in in_slot; V_t is
 * written to local slot buf_slot + (t-t0-1) % buf_len and, if keep_every > 0 and
 * (t-t0) % keep_every == 0, also to local slot keep_slot + (t-t0)/keep_every - 1.
 * FWD generates and stores the events; REFWD* replays the stored events.
 * BWD back-propagates t = t1 .. t0+1 with V_t in local slot buf_slot + (t-t0-1).
 * D2H copies local slot in_slot to remote slot remote_slot; H2D the reverse into keep_slot; both move
 * max(buf_len, 1) consecutive slots in one transfer.
 * ZERO clears local slot keep_slot (the initial state). */
typedef enum { SNN_OP_FWD = 0, SNN_OP_REFWD1 = 1, SNN_OP_REFWD2 = 2, SNN_OP_BWD = 3,
               SNN_OP_D2H = 4, SNN_OP_H2D = 5, SNN_OP_ZERO = 6 } snn_op_kind;
typedef struct {
  int32_t kind, t0, t1;
  int32_t in_slot, buf_slot, buf_len;
  int32_t keep_every, keep_slot, remote_slot;
} snn_op;
/* Writes up to max_ops operations to ops (may be NULL to query) and the totals.
 * Pure host function: usable without a GPU. */
snn_status snn_plan(int32_t T, const snn_ckpt* ckpt, snn_op* ops, int32_t max_ops, int32_t* n_ops,
                    int32_t* n_local_slots, int32_t* n_remote_slots);

/* ---- self-test of the bounded waits ---------------------------------------------------------
 * The cooperative kernels (forward and backward passes of small networks) wait for one another's results
 * by polling counters in device memory; every such wait gives up after a fixed number of polls, raises a
 * status bit and lets the kernel end, and the train step then returns SNN_ERR_DEVICE_TIMEOUT.  This call
 * runs that wait alone: one thread block waits, for at most poll_limit polls, for a count that nobody
 * publishes.  device_scratch: 256 bytes of device memory (overwritten).  Returns SNN_ERR_DEVICE_TIMEOUT
 * when the wait gave up as it must, SNN_OK if it did not, SNN_ERR_CUDA on a CUDA error.  The context
 * stays usable. */
snn_status snn_selftest_wait_timeout(void* device_scratch, uint32_t poll_limit, void* stream);

/* ---- spike compaction on its own ("Spike Generation": dense state -> sparse events) -----
 * For each of n_rows rows of n_words uint32 spike words (device), writes the ascending list
 * of set-bit indices to idx_out[row * capacity ..] (device) and its length to count_out[row]
 * (device).  Entries beyond capacity are dropped but still counted. */
snn_status snn_compact_spikes(const uint32_t* masks, int32_t n_rows, int32_t n_words, uint32_t* idx_out,
                              int32_t capacity, uint32_t* count_out, void* stream);

/* ---- where the last step left its events (for inspection) -------------------------------
 * layer 0 = input, 1..L = hidden.  List (layer, t, b), t = 1..T, is
 * pool[b * pool_capacity + offsets[t * B + b] .. offsets[(t+1) * B + b]).  Offsets are byte
 * offsets into device_ws. */
typedef struct {
  size_t offsets_off;  /* uint32 [(T+2)][B]                                   */
  size_t pool_off;     /* uint32 [B][pool_capacity] neuron indices            */
  size_t values_off;   /* fp32  [B][pool_capacity] (graded cell), else 0      */
  size_t pool_capacity;
  size_t mask_off;     /* uint32 [(T+1)][B][mask_words] (hidden layers), else 0 */
  int32_t mask_words;
} snn_event_layout;
snn_status snn_get_event_layout(const snn_net* net, int32_t layer, snn_event_layout* out);

#ifdef __cplusplus
}
#endif
#endif /* SNN_H_ */
