// Host-side schedule generator: the execution traces of the paper's Fig. 1 (forward,
// re-forward_1, re-forward_2, backward, loads and stores of remote checkpoints) written as
// a list of segment operations over numbered state slots.  No CUDA here.
//
// Slot counts against the paper's cost models (M_s = one dense state):
//   STANDARD  T + 1            Eq. 2: T states, plus the initial one
//   CHUNK     K + ceil(T/K)    Eq. 4: chunk buffer + checkpoints (the initial state is one)
//   REMOTE    K + 2            Eq. 6 has K + 1; the second staging slot lets the next load
//                              overlap the recomputation of the current segment
//   DOUBLE    K + R/K + 1      Eq. 11 has K + R/K; same extra staging slot
//   HIERARCHICAL  K + nb_local Eq. 9 exactly: no staging slot, the batch of the next nb_local
//                              checkpoints is fetched while the last segment of the current batch
//                              is back-propagated
#include <algorithm>
#include <cmath>
#include <vector>

#include "../../include/snn.h"

namespace {

struct Plan {
  std::vector<snn_op> ops;
  int n_local = 0, n_remote = 0;
};

snn_op make_op(int kind, int t0, int t1, int in_slot, int buf_slot, int buf_len, int keep_every,
               int keep_slot, int remote_slot) {
  snn_op o;
  o.kind = kind; o.t0 = t0; o.t1 = t1; o.in_slot = in_slot; o.buf_slot = buf_slot; o.buf_len = buf_len;
  o.keep_every = keep_every; o.keep_slot = keep_slot; o.remote_slot = remote_slot;
  return o;
}

int ceil_div(int a, int b) { return (a + b - 1) / b; }

bool build(int T, const snn_ckpt& ck, Plan& p) {
  auto zero = [&](int slot) { p.ops.push_back(make_op(SNN_OP_ZERO, 0, 0, -1, -1, 0, 0, slot, -1)); };
  auto d2h = [&](int slot, int r, int count = 1) { p.ops.push_back(make_op(SNN_OP_D2H, 0, 0, slot, -1, count, 0, -1, r)); };
  auto h2d = [&](int r, int slot, int count = 1) { p.ops.push_back(make_op(SNN_OP_H2D, 0, 0, -1, -1, count, 0, slot, r)); };
  if (ck.strategy == SNN_STANDARD) {
    p.n_local = T + 1;
    zero(0);
    p.ops.push_back(make_op(SNN_OP_FWD, 0, T, 0, 1, T, 0, -1, -1));
    p.ops.push_back(make_op(SNN_OP_BWD, 0, T, -1, 1, T, 0, -1, -1));
    return true;
  }
  const int K = ck.chunk_size;
  if (K < 1) return false;
  const int Kc = std::min(K, T);
  if (ck.strategy == SNN_CHUNK || ck.strategy == SNN_REMOTE) {
    const bool remote = ck.strategy == SNN_REMOTE;
    const int n_ck = ceil_div(T, K);
    // CHUNK: slots [0, n_ck) checkpoints, then the chunk buffer.  REMOTE: slots 0, 1 staging.
    const int buf = remote ? 2 : n_ck;
    p.n_local = buf + Kc;
    p.n_remote = remote ? n_ck : 0;
    auto ck_slot = [&](int c) { return remote ? c % 2 : c; };
    zero(ck_slot(0));
    if (remote) d2h(ck_slot(0), 0);
    for (int c = 0; c < n_ck; ++c) {
      const int t0 = c * K, t1 = std::min(T, t0 + K);
      const bool keep = t1 < T;  // a state at T is never a checkpoint
      p.ops.push_back(make_op(SNN_OP_FWD, t0, t1, ck_slot(c), buf, Kc, keep ? K : 0,
                              keep ? ck_slot(c + 1) : -1, -1));
      if (keep && remote) d2h(ck_slot(c + 1), c + 1);
    }
    if (remote) h2d(n_ck - 1, ck_slot(n_ck - 1));
    for (int c = n_ck - 1; c >= 0; --c) {
      const int t0 = c * K, t1 = std::min(T, t0 + K);
      if (remote && c > 0) h2d(c - 1, ck_slot(c - 1));  // prefetch the next segment's checkpoint
      p.ops.push_back(make_op(SNN_OP_REFWD1, t0, t1, ck_slot(c), buf, Kc, 0, -1, -1));
      p.ops.push_back(make_op(SNN_OP_BWD, t0, t1, -1, buf, Kc, 0, -1, -1));
    }
    return true;
  }
  if (ck.strategy == SNN_DOUBLE || ck.strategy == SNN_DOUBLE_LOCAL) {
    const int R = ck.remote_chunk_size;
    if (R < K || R % K != 0) return false;
    const int n_r = ceil_div(T, R);
    const int n_fine = ceil_div(std::min(R, T), K) - 1;  // local checkpoints besides the loaded one
    const int fine0 = 2, buf = 2 + n_fine;
    p.n_local = buf + Kc;
    p.n_remote = n_r;
    zero(0);
    d2h(0, 0);
    for (int r = 0; r < n_r; ++r) {
      const int t0 = r * R, t1 = std::min(T, t0 + R);
      const bool keep = t1 < T;
      p.ops.push_back(make_op(SNN_OP_FWD, t0, t1, r % 2, buf, Kc, keep ? R : 0, keep ? (r + 1) % 2 : -1, -1));
      if (keep) d2h((r + 1) % 2, r + 1);
    }
    h2d(n_r - 1, (n_r - 1) % 2);
    for (int r = n_r - 1; r >= 0; --r) {
      const int r0 = r * R, r1 = std::min(T, r0 + R);
      if (r > 0) h2d(r - 1, (r - 1) % 2);
      const int nf = ceil_div(r1 - r0, K);
      const int last_fine = r0 + (nf - 1) * K;
      if (nf > 1)  // re-forward_1 stops at the last local checkpoint of the segment
        p.ops.push_back(make_op(SNN_OP_REFWD1, r0, last_fine, r % 2, buf, Kc, K, fine0, -1));
      for (int f = nf - 1; f >= 0; --f) {
        const int t0 = r0 + f * K, t1 = std::min(r1, t0 + K);
        const int in = f == 0 ? r % 2 : fine0 + f - 1;
        p.ops.push_back(make_op(SNN_OP_REFWD2, t0, t1, in, buf, Kc, 0, -1, -1));
        p.ops.push_back(make_op(SNN_OP_BWD, t0, t1, -1, buf, Kc, 0, -1, -1));
      }
    }
    return true;
  }
  if (ck.strategy == SNN_HIERARCHICAL) {
    // Checkpoints every K steps, handled in batches of P = nb_local: checkpoint c lives in local slot
    // c % P.  Forward: a full batch that is not the last one goes to remote memory in one transfer;
    // the last batch never leaves.  Backward: batches in descending order; the previous batch is
    // fetched in one transfer right after the re-forward of the current batch's lowest checkpoint,
    // so the copy overlaps that segment's backward pass and needs no extra slot.
    const int P = std::max(1, std::min(ck.nb_local, ceil_div(T, K)));
    if (ck.nb_local < 1) return false;
    const int n_ck = ceil_div(T, K), n_b = ceil_div(n_ck, P);
    const int buf = P;
    p.n_local = P + Kc;
    p.n_remote = (n_b - 1) * P;
    zero(0);
    if (P == 1 && n_b > 1) d2h(0, 0, 1);   // a batch of one: the initial state is complete at once
    for (int c = 0; c < n_ck; ++c) {
      const int t0 = c * K, t1 = std::min(T, t0 + K);
      const bool keep = t1 < T;
      p.ops.push_back(make_op(SNN_OP_FWD, t0, t1, c % P, buf, Kc, keep ? K : 0, keep ? (c + 1) % P : -1, -1));
      // checkpoint c+1 completes batch (c+1)/P when it is that batch's last one
      if (keep && (c + 2) % P == 0 && (c + 1) / P < n_b - 1) d2h(0, ((c + 1) / P) * P, P);
    }
    for (int j = n_b - 1; j >= 0; --j) {
      const int c_lo = j * P, c_hi = std::min(n_ck, c_lo + P) - 1;
      for (int c = c_hi; c >= c_lo; --c) {
        const int t0 = c * K, t1 = std::min(T, t0 + K);
        p.ops.push_back(make_op(SNN_OP_REFWD1, t0, t1, c % P, buf, Kc, 0, -1, -1));
        if (c == c_lo && j > 0) h2d((j - 1) * P, 0, P);
        p.ops.push_back(make_op(SNN_OP_BWD, t0, t1, -1, buf, Kc, 0, -1, -1));
      }
    }
    return true;
  }
  return false;
}

}  // namespace

extern "C" snn_status snn_plan(int32_t T, const snn_ckpt* ckpt, snn_op* ops, int32_t max_ops, int32_t* n_ops,
                               int32_t* n_local_slots, int32_t* n_remote_slots) {
  if (!ckpt || T < 1) return SNN_ERR_INVALID_ARG;
  Plan p;
  if (!build(T, *ckpt, p)) return SNN_ERR_INVALID_ARG;
  if (n_ops) *n_ops = (int32_t)p.ops.size();
  if (n_local_slots) *n_local_slots = p.n_local;
  if (n_remote_slots) *n_remote_slots = p.n_remote;
  if (ops) {
    if (max_ops < (int32_t)p.ops.size()) return SNN_ERR_INVALID_ARG;
    std::copy(p.ops.begin(), p.ops.end(), ops);
  }
  return SNN_OK;
}

// Hyper-parameter rules of the paper's Hyperparameter Study (see snn.h).
extern "C" snn_status snn_suggest_ckpt(const snn_net* net, int32_t T, int32_t B, int32_t strategy,
                                       size_t device_budget_bytes, float max_activity, snn_ckpt* out) {
  if (!out || T < 1) return SNN_ERR_INVALID_ARG;
  auto isqrt = [](int x) { return std::max(1, (int)std::lround(std::sqrt((double)x))); };
  snn_ckpt c{strategy, 0, 0, 0};
  switch (strategy) {
    case SNN_STANDARD: break;
    case SNN_CHUNK: c.chunk_size = isqrt(T); break;
    case SNN_HIERARCHICAL:
      c.chunk_size = isqrt(T);
      c.nb_local = isqrt(ceil_div(T, c.chunk_size));
      break;
    case SNN_DOUBLE:
    case SNN_DOUBLE_LOCAL: {
      int R = 256;
      if (T < 1024) { R = 4; while (R * 2 <= std::max(4, T / 4) && R < 256) R *= 2; }
      c.chunk_size = isqrt(R);
      while (R % c.chunk_size != 0) ++c.chunk_size;   // R is a power of two: ends at a power of two
      c.remote_chunk_size = R;
      break;
    }
    case SNN_REMOTE: {
      c.chunk_size = isqrt(T);
      if (device_budget_bytes > 0) {
        if (!net || B < 1) return SNN_ERR_INVALID_ARG;
        int lo = 0, hi = T;   // largest K in [1, T] whose workspace fits; 0 = none fits
        while (lo < hi) {
          const int mid = (lo + hi + 1) / 2;
          snn_ckpt q{SNN_REMOTE, mid, 0, 0};
          size_t dev = 0, pin = 0;
          const bool ok = snn_workspace_query(net, T, B, &q, max_activity, &dev, &pin) == SNN_OK &&
                          dev <= device_budget_bytes;
          if (ok) lo = mid; else hi = mid - 1;
        }
        if (lo < 1) return SNN_ERR_WORKSPACE_TOO_SMALL;
        c.chunk_size = lo;
      }
      break;
    }
    default: return SNN_ERR_INVALID_ARG;
  }
  *out = c;
  return SNN_OK;
}
