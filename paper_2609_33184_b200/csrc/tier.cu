// Commit-aware KV tiering (Section 4.1): Sealed History [0, H) in pinned host memory, Active
// Tail [H, C) on the GPU, the speculative frontier past C never leaves the GPU.  Committed KV
// accumulates in the tail; older contiguous blocks are offloaded in batches: the migration end
// point is Eq. 9, E = max{H, g * floor(max(0, C - T) / g)}; [H, E) is copied asynchronously and
// the history boundary advances to E only after the copy is confirmed.  Rejected candidates
// only ever change the region past C, so nothing on the host is rolled back.
//
// Host code only: boundary arithmetic, copy submission, confirmation.  The tail lives in one of
// two device buffers [B, H_kv, tail_capacity, d] (token t of request b at index t - H_b); when
// boundaries advance the surviving tail [E, C) is copied to the front of the other buffer and
// the buffers swap, for all requests at once (one tensor view serves the whole batch).
#include <cstring>
#include <new>

#include "ss_internal.h"

struct ss_tier {
  ss_tier_config cfg;
  void* host_hist[1024];
  int64_t host_cap[1024];
  void* tail_k[2];
  void* tail_v[2];
  int32_t* len_dev;     // device [B]: tail length C - H (valid_len of the tail chunk, gather offset)
  int32_t* len_host;    // pinned [4][B]: a ring; a slot is rewritten only after the copy that read it
                        // has finished (one event per slot, waited for before reuse)
  int len_slot;
  cudaEvent_t ev_len[4];
  bool len_used[4];
  int32_t H[1024], C[1024], E[1024];
  int cur;              // buffer holding the tail
  bool pending;         // a migration is in flight
  cudaEvent_t ev_copied;
  int64_t d2h_bytes;
  int32_t migrations;
};

namespace {
int32_t endpoint(int32_t H, int32_t C, int32_t T, int32_t g) {  // Eq. 9
  const int32_t over = C - T > 0 ? C - T : 0;
  const int32_t e = g * (over / g);
  return e > H ? e : H;
}
}  // namespace

extern "C" {

ss_status ss_tier_create(ss_tier** out, const ss_tier_config* cfg, void* const* host_hist,
                         const int64_t* host_capacity_tokens, void* tail_k0, void* tail_v0,
                         void* tail_k1, void* tail_v1, int32_t* len_dev, int32_t* len_host) {
  if (!out || !cfg || !host_hist || !host_capacity_tokens || !tail_k0 || !tail_v0 || !tail_k1 ||
      !tail_v1 || !len_dev || !len_host)
    return SS_ERR_ARG;
  if (cfg->B <= 0 || cfg->B > 1024 || cfg->H_kv <= 0 || (cfg->d != 64 && cfg->d != 128) ||
      cfg->L_c <= 0 || cfg->tail_target < 0 || cfg->granularity <= 0 || cfg->tail_capacity <= 0)
    return SS_ERR_SHAPE;
  // the tail must hold T + g committed tokens plus a round of accepted candidates
  if (cfg->tail_capacity < cfg->tail_target + cfg->granularity) return SS_ERR_CAPACITY;
  ss_tier* t = new (std::nothrow) ss_tier();
  if (!t) return SS_ERR_ARG;
  memset(t, 0, sizeof(*t));
  t->cfg = *cfg;
  for (int b = 0; b < cfg->B; ++b) {
    if (!host_hist[b] || host_capacity_tokens[b] % cfg->L_c) {
      delete t;
      return SS_ERR_ARG;
    }
    t->host_hist[b] = host_hist[b];
    t->host_cap[b] = host_capacity_tokens[b];
  }
  t->tail_k[0] = tail_k0;
  t->tail_v[0] = tail_v0;
  t->tail_k[1] = tail_k1;
  t->tail_v[1] = tail_v1;
  t->len_dev = len_dev;
  t->len_host = len_host;
  bool ok = cudaEventCreateWithFlags(&t->ev_copied, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; i < 4 && ok; ++i)
    ok = cudaEventCreateWithFlags(&t->ev_len[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    if (t->ev_copied) cudaEventDestroy(t->ev_copied);
    for (int i = 0; i < 4; ++i)
      if (t->ev_len[i]) cudaEventDestroy(t->ev_len[i]);
    delete t;
    return SS_ERR_CUDA;
  }
  *out = t;
  return SS_OK;
}

ss_status ss_tier_destroy(ss_tier* t) {
  if (!t) return SS_ERR_ARG;
  cudaEventDestroy(t->ev_copied);
  for (int i = 0; i < 4; ++i) cudaEventDestroy(t->ev_len[i]);
  delete t;
  return SS_OK;
}

// Publish the tail lengths C - H to the device through the next slot of the pinned ring.
static ss_status publish_lengths(ss_tier* t, cudaStream_t s) {
  t->len_slot = (t->len_slot + 1) & 3;
  const int i = t->len_slot;
  // the copy that last read this slot (four publishes ago) must have finished
  if (t->len_used[i] && cudaEventSynchronize(t->ev_len[i]) != cudaSuccess) return SS_ERR_CUDA;
  int32_t* slot = t->len_host + (size_t)i * t->cfg.B;
  for (int b = 0; b < t->cfg.B; ++b) slot[b] = t->C[b] - t->H[b];
  if (cudaMemcpyAsync(t->len_dev, slot, sizeof(int32_t) * t->cfg.B, cudaMemcpyHostToDevice, s) !=
      cudaSuccess)
    return SS_ERR_CUDA;
  if (cudaEventRecord(t->ev_len[i], s) != cudaSuccess) return SS_ERR_CUDA;
  t->len_used[i] = true;
  return SS_OK;
}

ss_status ss_tier_reset(ss_tier* t, const int32_t* H, const int32_t* C, void* stream) {
  if (!t || !H || !C) return SS_ERR_ARG;
  if (t->pending) return SS_ERR_STATE;
  for (int b = 0; b < t->cfg.B; ++b) {
    if (H[b] < 0 || H[b] % t->cfg.granularity || C[b] < H[b] || C[b] - H[b] > t->cfg.tail_capacity ||
        H[b] > t->host_cap[b])
      return SS_ERR_ARG;
  }
  for (int b = 0; b < t->cfg.B; ++b) {
    t->H[b] = H[b];
    t->C[b] = C[b];
    t->E[b] = H[b];
  }
  t->cur = 0;
  return publish_lengths(t, (cudaStream_t)stream);
}

ss_status ss_tier_get(ss_tier* t, int32_t* H, int32_t* C, int32_t* pending_E, int32_t* cur_buffer) {
  if (!t) return SS_ERR_ARG;
  for (int b = 0; b < t->cfg.B; ++b) {
    if (H) H[b] = t->H[b];
    if (C) C[b] = t->C[b];
    if (pending_E) pending_E[b] = t->pending ? t->E[b] : t->H[b];
  }
  if (cur_buffer) *cur_buffer = t->cur;
  return SS_OK;
}

ss_status ss_tier_tail(ss_tier* t, ss_tensor* K, ss_tensor* V, const int32_t** tail_len_dev) {
  if (!t || !K || !V) return SS_ERR_ARG;
  const int64_t row = t->cfg.d, cap = t->cfg.tail_capacity;
  *K = {t->tail_k[t->cur], (int64_t)t->cfg.H_kv * cap * row, cap * row, row};
  *V = {t->tail_v[t->cur], (int64_t)t->cfg.H_kv * cap * row, cap * row, row};
  if (tail_len_dev) *tail_len_dev = t->len_dev;
  return SS_OK;
}

ss_status ss_tier_commit(ss_tier* t, const int32_t* cnt, void* stream) {
  if (!t || !cnt) return SS_ERR_ARG;
  for (int b = 0; b < t->cfg.B; ++b)
    if (cnt[b] < 0 || t->C[b] + cnt[b] - t->H[b] > t->cfg.tail_capacity) return SS_ERR_CAPACITY;
  for (int b = 0; b < t->cfg.B; ++b) t->C[b] += cnt[b];
  return publish_lengths(t, (cudaStream_t)stream);
}

ss_status ss_tier_migrate(ss_tier* t, void* stream, int32_t* n_requests) {
  if (!t) return SS_ERR_ARG;
  if (t->pending) return SS_ERR_STATE;  // one migration in flight at a time
  cudaStream_t s = (cudaStream_t)stream;
  const ss_tier_config& c = t->cfg;
  const size_t esz = 2;
  const int64_t cap = c.tail_capacity;
  int moved = 0;
  // every end point is checked against its host capacity before the first copy is enqueued
  for (int b = 0; b < c.B; ++b)
    if (endpoint(t->H[b], t->C[b], c.tail_target, c.granularity) > t->host_cap[b]) return SS_ERR_CAPACITY;
  for (int b = 0; b < c.B; ++b) {
    const int32_t E = endpoint(t->H[b], t->C[b], c.tail_target, c.granularity);
    t->E[b] = E;
    if (E <= t->H[b]) continue;
    ++moved;
    // [H, E) -> host chunk blocks [chunk][K|V][H_kv][L_c][d]; one 2-D copy per chunk segment and K|V
    for (int32_t tok = t->H[b]; tok < E;) {
      const int32_t j = tok / c.L_c, r = tok % c.L_c;
      const int32_t n = (E - tok < c.L_c - r) ? E - tok : c.L_c - r;
      for (int kv = 0; kv < 2; ++kv) {
        const uint16_t* src = (const uint16_t*)(kv ? t->tail_v[t->cur] : t->tail_k[t->cur]) +
                              ((int64_t)b * c.H_kv * cap + (tok - t->H[b])) * c.d;
        uint16_t* dst = (uint16_t*)t->host_hist[b] +
                        ((int64_t)j * 2 * c.H_kv + (int64_t)kv * c.H_kv) * c.L_c * c.d + (int64_t)r * c.d;
        if (cudaMemcpy2DAsync(dst, (size_t)c.L_c * c.d * esz, src, (size_t)cap * c.d * esz,
                              (size_t)n * c.d * esz, c.H_kv, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
          // Copies of this call may already be in flight.  Let them finish and leave every
          // boundary where it was: the host blocks they wrote lie past H and are written
          // again by the next migration.
          cudaStreamSynchronize(s);
          for (int q = 0; q < c.B; ++q) t->E[q] = t->H[q];
          return SS_ERR_CUDA;
        }
        t->d2h_bytes += (int64_t)n * c.d * esz * c.H_kv;
      }
      tok += n;
    }
  }
  if (n_requests) *n_requests = moved;
  if (!moved) return SS_OK;
  if (cudaEventRecord(t->ev_copied, s) != cudaSuccess) return SS_ERR_CUDA;
  t->pending = true;
  ++t->migrations;
  return SS_OK;
}

ss_status ss_tier_poll(ss_tier* t, int32_t wait, void* stream, int32_t* advanced) {
  if (!t) return SS_ERR_ARG;
  if (advanced) *advanced = 0;
  if (!t->pending) return SS_OK;
  if (wait) {
    if (cudaEventSynchronize(t->ev_copied) != cudaSuccess) return SS_ERR_CUDA;
  } else {
    const cudaError_t q = cudaEventQuery(t->ev_copied);
    if (q == cudaErrorNotReady) return SS_OK;  // not confirmed: boundaries stay where they are
    if (q != cudaSuccess) return SS_ERR_CUDA;
  }
  // the copies are confirmed: advance H, move the surviving tails to the other buffer
  cudaStream_t s = (cudaStream_t)stream;
  const ss_tier_config& c = t->cfg;
  const size_t esz = 2, pitch = (size_t)c.tail_capacity * c.d * esz;
  const int nxt = t->cur ^ 1;
  for (int b = 0; b < c.B; ++b) {
    const int32_t keep = t->C[b] - t->E[b];
    if (keep > 0) {
      for (int kv = 0; kv < 2; ++kv) {
        const uint16_t* src = (const uint16_t*)(kv ? t->tail_v[t->cur] : t->tail_k[t->cur]) +
                              ((int64_t)b * c.H_kv * c.tail_capacity + (t->E[b] - t->H[b])) * c.d;
        uint16_t* dst = (uint16_t*)(kv ? t->tail_v[nxt] : t->tail_k[nxt]) +
                        (int64_t)b * c.H_kv * c.tail_capacity * c.d;
        if (cudaMemcpy2DAsync(dst, pitch, src, pitch, (size_t)keep * c.d * esz, c.H_kv,
                              cudaMemcpyDeviceToDevice, s) != cudaSuccess)
          return SS_ERR_CUDA;
      }
    }
    t->H[b] = t->E[b];
  }
  t->cur = nxt;
  t->pending = false;
  if (advanced) *advanced = 1;
  return publish_lengths(t, s);
}

int64_t ss_tier_d2h_bytes(ss_tier* t) { return t ? t->d2h_bytes : 0; }

}  // extern "C"
