// Streamed rounds: pinned-host history -> two device staging buffers on a copy stream, chunk
// attention on an attention stream, hand-off by events (Section 4.2, pipelined KV transfers and
// prefetching).  While the attention stream works on buffer A, buffer B receives the next fill;
// a fill carries `batch_chunks` adjacent chunks (a transfer batch).  ss_stream_layers runs
// several layers back to back: with cross-layer prefetch the copy stream starts the next
// layer's first fills as soon as a staging buffer frees, without waiting for the current
// layer's remaining attention, finalize and commit.
#include <chrono>
#include <cstring>

#include "ss_internal.h"

namespace ss {
struct PipeRes {
  cudaStream_t copy_stream, attn_stream;
  cudaEvent_t *ev_ready, *ev_free, ev_t0, ev_t1;
};
cudaError_t ctx_pipeline(ss_ctx* c, PipeRes* out);
int ctx_dims(ss_ctx* c, int* H_q, int* H_kv, int* d);
void ctx_set_cuda_error(ss_ctx* c, cudaError_t e);
void ctx_pipeline_mode(ss_ctx* c, bool on);
bool ctx_round_open(ss_ctx* c);
cudaEvent_t* ctx_timing_events(ss_ctx* c, int n);
void ctx_set_stream_times(ss_ctx* c, int64_t round_ns, int64_t transfer_ns, int64_t chunk_ns, int64_t tail_ns);
void ctx_pipeline_drain(ss_ctx* c);
}  // namespace ss

#define SS_CK(expr)                          \
  do {                                       \
    cudaError_t e_ = (expr);                 \
    if (e_ != cudaSuccess) {                 \
      ss::ctx_set_cuda_error(ctx, e_);       \
      return SS_ERR_CUDA;                    \
    }                                        \
  } while (0)
#define SS_ST(expr)                  \
  do {                               \
    ss_status s_ = (expr);           \
    if (s_ != SS_OK) return s_;      \
  } while (0)

namespace {

struct LayerCounts {
  int64_t h2d = 0, d2h = 0;
  int copies = 0, calls = 0, fills = 0;
  // phase timing (ss_stream_round with SS_FLAG_STREAM_TIMING): ev[0] = last history copy done,
  // ev[1] = start of the local / finalize / commit tail, ev[2 + 2i], ev[3 + 2i] around chunk call i
  cudaEvent_t* ev = nullptr;
  int ev_cap = 0, timed_calls = 0;
};

// A chunk call of the streamed round, with an event pair around it when the round is timed.
ss_status timed_chunk(ss_ctx* ctx, LayerCounts* cnt, cudaStream_t s, ss_tensor K, ss_tensor V, int32_t L_c,
                      const int32_t* vl_dev, const int32_t* vl_host) {
  const bool timed = cnt->ev && 3 + 2 * cnt->timed_calls < cnt->ev_cap;
  if (timed) SS_CK(cudaEventRecord(cnt->ev[2 + 2 * cnt->timed_calls], s));
  SS_ST(vl_host ? ss_verify_chunk_hinted(ctx, K, V, L_c, vl_dev, vl_host, s)
                : ss_verify_chunk(ctx, K, V, L_c, vl_dev, s));
  if (timed) {
    SS_CK(cudaEventRecord(cnt->ev[3 + 2 * cnt->timed_calls], s));
    ++cnt->timed_calls;
  }
  ++cnt->calls;
  return SS_OK;
}

ss_status validate_desc(ss_ctx* ctx, const ss_stream_desc* d, int* n_fills_out) {
  if (!d || !d->hist || !d->hist_len) return SS_ERR_ARG;
  if (d->B <= 0 || d->T_q <= 0 || d->L_c <= 0 || d->batch_chunks <= 0) return SS_ERR_ARG;
  if (!d->stage_k[0] || !d->stage_k[1]) return SS_ERR_ARG;
  if (!d->stage_fused && (!d->stage_v[0] || !d->stage_v[1])) return SS_ERR_ARG;
  if (!d->valid_len_host || !d->valid_len_dev) return SS_ERR_ARG;
  if (!d->copy_only && (!d->Q.ptr || !d->K_loc.ptr || !d->V_loc.ptr || !d->O)) return SS_ERR_ARG;
  int H_q, H_kv, hd;
  if (d->B > ss::ctx_dims(ctx, &H_q, &H_kv, &hd)) return SS_ERR_SHAPE;
  int max_len = 0;
  for (int b = 0; b < d->B; ++b) {
    if (d->hist_len[b] < 0 || (d->hist_len[b] > 0 && !d->hist[b])) return SS_ERR_ARG;
    if (d->hist_len[b] > max_len) max_len = d->hist_len[b];
  }
  const int n_chunks = (max_len + d->L_c - 1) / d->L_c;
  const int n_fills = (n_chunks + d->batch_chunks - 1) / d->batch_chunks;
  // the valid-length scratch holds one row of B entries per chunk call
  const int n_calls = d->stage_fused == 2 ? n_fills * d->batch_chunks : n_fills;
  if (n_calls > d->scratch_fills) return SS_ERR_CAPACITY;
  if (d->stage_fused < 0 || d->stage_fused > 2) return SS_ERR_ARG;
  *n_fills_out = n_fills;
  return SS_OK;
}

// Enqueue one layer's round on the two streams; synchronises nothing.  `fill_base` numbers the
// fills across layers so that consecutive layers keep alternating the two staging buffers.
// restore_k != null: the restore-then-verify baseline - the whole history of the layer is
// copied into restore_k / restore_v first and only then attended to.
ss_status enqueue_layer(ss_ctx* ctx, const ss_stream_desc* d, const ss::PipeRes& r, int n_fills,
                        int fill_base, void* restore_k, void* restore_v, int64_t restore_tokens,
                        LayerCounts* cnt) {
  int H_q, H_kv, hd;
  ss::ctx_dims(ctx, &H_q, &H_kv, &hd);
  const int B = d->B, L_c = d->L_c, bc = d->batch_chunks;
  const bool restore = restore_k != nullptr;
  // K and V of a block next to each other in one device buffer ([B][K|V][H_kv][Ls][d]): the
  // staging slots with stage_fused, the restore buffer when restore_v is null
  const bool fused = restore ? restore_v == nullptr : d->stage_fused != 0;
  // block-major staging: a slot is [B][bc][K|V][H_kv][L_c][d], the host's own block order, so a
  // fill moves up to bc adjacent blocks of a request with ONE copy and is consumed by bc chunk
  // calls of L_c tokens
  const bool blocks = !restore && d->stage_fused == 2;
  const int64_t Ls = restore ? restore_tokens : (blocks ? L_c : (int64_t)bc * L_c);  // tokens per device row
  // with stage_fused == 2 every chunk call takes L_c tokens (also on the restored copy)
  const bool per_chunk = d->stage_fused == 2;
  const int rows_vl = per_chunk ? n_fills * bc : n_fills;   // rows of the valid-length scratch
  const int64_t span = per_chunk ? L_c : (int64_t)bc * L_c; // tokens one scratch row covers
  if (restore && (int64_t)n_fills * bc * L_c > restore_tokens) return SS_ERR_CAPACITY;
  int64_t max_len = 0;
  for (int b = 0; b < B; ++b) max_len = d->hist_len[b] > max_len ? d->hist_len[b] : max_len;

  for (int f = 0; f < rows_vl; ++f)
    for (int b = 0; b < B; ++b) {
      int64_t v = (int64_t)d->hist_len[b] - (int64_t)f * span;
      v = v < 0 ? 0 : (v > span ? span : v);
      d->valid_len_host[f * B + b] = (int32_t)v;
    }
  if (rows_vl)
    SS_CK(cudaMemcpyAsync(d->valid_len_dev, d->valid_len_host, sizeof(int32_t) * rows_vl * B,
                          cudaMemcpyHostToDevice, r.copy_stream));
  if (!d->copy_only) {
    SS_ST(ss_verify_begin(ctx, d->Q, B, d->T_q, d->scale, r.attn_stream));
    if (d->tail_K.ptr) {  // on-GPU Active Tail: no copy, runs while the first fills arrive
      if (!d->tail_V.ptr || d->tail_Lc <= 0) return SS_ERR_ARG;
      SS_ST(timed_chunk(ctx, cnt, r.attn_stream, d->tail_K, d->tail_V, d->tail_Lc, d->tail_len, nullptr));
    }
  }

  const size_t esz = 2;
  const int64_t head_elems = (int64_t)L_c * hd;          // one head row of a host block
  const int64_t block_elems = 2 * (int64_t)H_kv * head_elems;
  for (int f = 0; f < n_fills; ++f) {
    const int buf = (fill_base + f) & 1;
    if (!restore && fill_base + f >= 2) SS_CK(cudaStreamWaitEvent(r.copy_stream, r.ev_free[buf], 0));
    if (blocks) {
      int last_chunk = -1;  // last chunk index of this fill that holds tokens of any request
      for (int b = 0; b < B; ++b) {
        const int64_t j0 = (int64_t)f * bc;
        const int64_t rem = (int64_t)d->hist_len[b] - j0 * L_c;
        if (rem <= 0) continue;
        int64_t nfull = rem / L_c;
        if (nfull > bc) nfull = bc;
        const int64_t part = nfull < bc ? rem - nfull * L_c : 0;  // tokens of a partial block
        const uint16_t* src = (const uint16_t*)d->hist[b] + j0 * block_elems;
        uint16_t* dst = (uint16_t*)d->stage_k[buf] + (int64_t)b * bc * block_elems;
        if (nfull > 0) {
          SS_CK(cudaMemcpyAsync(dst, src, (size_t)(nfull * block_elems) * esz, cudaMemcpyHostToDevice,
                                r.copy_stream));
          cnt->h2d += nfull * block_elems * (int64_t)esz;
          ++cnt->copies;
        }
        if (part > 0) {
          SS_CK(cudaMemcpy2DAsync(dst + nfull * block_elems, (size_t)head_elems * esz,
                                  src + nfull * block_elems, (size_t)head_elems * esz,
                                  (size_t)part * hd * esz, 2 * H_kv, cudaMemcpyHostToDevice,
                                  r.copy_stream));
          cnt->h2d += 2 * (int64_t)H_kv * part * hd * esz;
          ++cnt->copies;
        }
        const int lastb = (int)(j0 + nfull + (part > 0 ? 1 : 0)) - 1;
        if (lastb > last_chunk) last_chunk = lastb;
      }
      SS_CK(cudaEventRecord(r.ev_ready[buf], r.copy_stream));
      SS_CK(cudaStreamWaitEvent(r.attn_stream, r.ev_ready[buf], 0));
      if (!d->copy_only) {
        for (int jj = 0; jj < bc && f * bc + jj <= last_chunk; ++jj) {
          const int j = f * bc + jj;
          const uint16_t* kb = (const uint16_t*)d->stage_k[buf] + (int64_t)jj * block_elems;
          ss_tensor K = {kb, (int64_t)bc * block_elems, head_elems, hd};
          ss_tensor V = {kb + (int64_t)H_kv * head_elems, (int64_t)bc * block_elems, head_elems, hd};
          SS_ST(timed_chunk(ctx, cnt, r.attn_stream, K, V, L_c, d->valid_len_dev + (int64_t)j * B,
                            d->valid_len_host + (int64_t)j * B));
        }
      }
      SS_CK(cudaEventRecord(r.ev_free[buf], r.attn_stream));
      continue;
    }
    for (int jj = 0; jj < bc; ++jj) {
      const int j = f * bc + jj;
      for (int b = 0; b < B; ++b) {
        int64_t v = (int64_t)d->hist_len[b] - (int64_t)j * L_c;
        if (v <= 0) continue;
        if (v > L_c) v = L_c;
        const uint16_t* src = (const uint16_t*)d->hist[b] + (int64_t)j * block_elems;
        if (fused) {
          // K and V of the block in one copy: the staging buffer keeps the host block's order
          uint16_t* dst = (restore ? (uint16_t*)restore_k + (int64_t)j * L_c * hd
                                   : (uint16_t*)d->stage_k[buf] + (int64_t)jj * L_c * hd) +
                          (int64_t)b * 2 * H_kv * Ls * hd;
          if (v == L_c && Ls == L_c) {
            SS_CK(cudaMemcpyAsync(dst, src, (size_t)block_elems * esz, cudaMemcpyHostToDevice,
                                  r.copy_stream));
          } else {
            SS_CK(cudaMemcpy2DAsync(dst, (size_t)Ls * hd * esz, src, (size_t)head_elems * esz,
                                    (size_t)v * hd * esz, 2 * H_kv, cudaMemcpyHostToDevice,
                                    r.copy_stream));
          }
          cnt->h2d += 2 * (int64_t)H_kv * v * hd * esz;
          ++cnt->copies;
          continue;
        }
        for (int kv = 0; kv < 2; ++kv) {
          uint16_t* base = restore ? (uint16_t*)(kv ? restore_v : restore_k)
                                   : (uint16_t*)(kv ? d->stage_v[buf] : d->stage_k[buf]);
          const int64_t tok = restore ? (int64_t)j * L_c : (int64_t)jj * L_c;
          uint16_t* dst = base + ((int64_t)b * H_kv * Ls + tok) * hd;
          const uint16_t* s = src + (int64_t)kv * H_kv * head_elems;
          if (v == L_c && Ls == L_c) {
            SS_CK(cudaMemcpyAsync(dst, s, (size_t)H_kv * head_elems * esz, cudaMemcpyHostToDevice,
                                  r.copy_stream));
          } else {
            SS_CK(cudaMemcpy2DAsync(dst, (size_t)Ls * hd * esz, s, (size_t)head_elems * esz,
                                    (size_t)v * hd * esz, H_kv, cudaMemcpyHostToDevice,
                                    r.copy_stream));
          }
          cnt->h2d += (int64_t)H_kv * v * hd * esz;
          ++cnt->copies;
        }
      }
    }
    if (restore) continue;  // attention starts after the last copy of the layer
    SS_CK(cudaEventRecord(r.ev_ready[buf], r.copy_stream));
    SS_CK(cudaStreamWaitEvent(r.attn_stream, r.ev_ready[buf], 0));
    if (!d->copy_only) {
      ss_tensor K = {d->stage_k[buf], (int64_t)H_kv * Ls * hd, Ls * hd, hd};
      ss_tensor V = {d->stage_v[buf], (int64_t)H_kv * Ls * hd, Ls * hd, hd};
      if (fused) {
        K.stride_b = V.stride_b = 2 * (int64_t)H_kv * Ls * hd;
        V.ptr = (const uint16_t*)d->stage_k[buf] + (int64_t)H_kv * Ls * hd;
      }
      SS_ST(timed_chunk(ctx, cnt, r.attn_stream, K, V, (int32_t)Ls, d->valid_len_dev + (int64_t)f * B,
                        d->valid_len_host + (int64_t)f * B));
    }
    SS_CK(cudaEventRecord(r.ev_free[buf], r.attn_stream));
  }
  if (restore || n_fills == 0) {
    // the attention stream follows the copy stream (whole history restored / nothing to stream)
    SS_CK(cudaEventRecord(r.ev_ready[0], r.copy_stream));
    SS_CK(cudaStreamWaitEvent(r.attn_stream, r.ev_ready[0], 0));
  }
  if (restore && !d->copy_only) {
    for (int f = 0; f < rows_vl; ++f) {  // the streamed path's chunk calls, on the restored copy
      const int64_t tok = (int64_t)f * span;
      if (per_chunk && tok >= max_len) break;
      ss_tensor K = {(uint16_t*)restore_k + tok * hd, (int64_t)H_kv * Ls * hd, Ls * hd, hd};
      ss_tensor V = {(uint16_t*)restore_v + tok * hd, (int64_t)H_kv * Ls * hd, Ls * hd, hd};
      if (fused) {
        K.stride_b = V.stride_b = 2 * (int64_t)H_kv * Ls * hd;
        V.ptr = (const uint16_t*)restore_k + (int64_t)H_kv * Ls * hd + tok * hd;
      }
      SS_ST(timed_chunk(ctx, cnt, r.attn_stream, K, V, (int32_t)span, d->valid_len_dev + (int64_t)f * B,
                        d->valid_len_host + (int64_t)f * B));
    }
  }
  cnt->fills += n_fills;
  if (cnt->ev) {
    SS_CK(cudaEventRecord(cnt->ev[0], r.copy_stream));   // the last history copy is behind this
    SS_CK(cudaEventRecord(cnt->ev[1], r.attn_stream));   // the tail starts here
  }
  if (!d->copy_only) {
    SS_ST(ss_verify_local(ctx, d->K_loc, d->V_loc, d->T_q, d->mask_kind, d->mask_bits, r.attn_stream));
    SS_ST(ss_verify_finalize(ctx, d->O, d->LSE, r.attn_stream));
    if (d->accept_idx) {
      if (!d->accept_cnt || !d->zero_off || !d->commit_k || !d->commit_v) return SS_ERR_ARG;
      const int64_t row = hd, tl = d->commit_cap > 0 ? d->commit_cap : d->T_q;
      ss_tensor Kd = {d->commit_k, (int64_t)H_kv * tl * row, tl * row, row};
      ss_tensor Vd = {d->commit_v, (int64_t)H_kv * tl * row, tl * row, row};
      SS_ST(ss_commit_gather(ctx, d->K_loc, d->V_loc, B, d->T_q, d->accept_idx, d->accept_cnt, Kd, Vd,
                             (int32_t)tl, d->zero_off, r.attn_stream));
      const size_t bytes = (size_t)B * H_kv * tl * row * esz;
      if (d->host_commit_k) {
        SS_CK(cudaMemcpyAsync(d->host_commit_k, d->commit_k, bytes, cudaMemcpyDeviceToHost, r.attn_stream));
        cnt->d2h += bytes;
      }
      if (d->host_commit_v) {
        SS_CK(cudaMemcpyAsync(d->host_commit_v, d->commit_v, bytes, cudaMemcpyDeviceToHost, r.attn_stream));
        cnt->d2h += bytes;
      }
    }
    if (d->O_host) {
      const size_t bytes = (size_t)B * H_q * d->T_q * hd * esz;
      SS_CK(cudaMemcpyAsync(d->O_host, d->O, bytes, cudaMemcpyDeviceToHost, r.attn_stream));
      cnt->d2h += bytes;
    }
    if (d->LSE_host && d->LSE) {
      const size_t bytes = (size_t)B * H_q * d->T_q * sizeof(float);
      SS_CK(cudaMemcpyAsync(d->LSE_host, d->LSE, bytes, cudaMemcpyDeviceToHost, r.attn_stream));
      cnt->d2h += bytes;
    }
  }
  return SS_OK;
}

void fill_stats(ss_stream_stats* st, const LayerCounts& c, float ms_device, double ms_total) {
  if (!st) return;
  st->ms_device = ms_device;
  st->ms_total = ms_total;
  st->h2d_bytes = c.h2d;
  st->d2h_bytes = c.d2h;
  st->chunk_calls = c.calls;
  st->copies = c.copies;
}

ss_status stream_round_impl(ss_ctx* ctx, const ss_stream_desc* d, ss_stream_stats* stats) {
  int n_fills = 0;
  SS_ST(validate_desc(ctx, d, &n_fills));
  ss::PipeRes r;
  SS_CK(ss::ctx_pipeline(ctx, &r));
  const auto wall0 = std::chrono::steady_clock::now();
  SS_CK(cudaEventRecord(r.ev_t0, r.copy_stream));
  LayerCounts cnt;
  // one event pair per chunk call (a fill of the block-major layout is batch_chunks calls, the
  // Active Tail one more) plus the two phase marks
  cnt.ev_cap = 2 + 2 * (n_fills * d->batch_chunks + 1);
  cnt.ev = ss::ctx_timing_events(ctx, cnt.ev_cap);
  SS_ST(enqueue_layer(ctx, d, r, n_fills, 0, nullptr, nullptr, 0, &cnt));
  SS_CK(cudaEventRecord(r.ev_t1, r.attn_stream));
  SS_CK(cudaEventSynchronize(r.ev_t1));
  SS_CK(cudaStreamSynchronize(r.copy_stream));
  float ms = 0.f;
  SS_CK(cudaEventElapsedTime(&ms, r.ev_t0, r.ev_t1));
  if (cnt.ev) {
    float t = 0.f, transfer = 0.f, tail = 0.f;
    double chunk = 0.0;
    SS_CK(cudaEventElapsedTime(&transfer, r.ev_t0, cnt.ev[0]));
    SS_CK(cudaEventElapsedTime(&tail, cnt.ev[1], r.ev_t1));
    for (int i = 0; i < cnt.timed_calls; ++i) {
      SS_CK(cudaEventElapsedTime(&t, cnt.ev[2 + 2 * i], cnt.ev[3 + 2 * i]));
      chunk += t;
    }
    ss::ctx_set_stream_times(ctx, (int64_t)(ms * 1e6), (int64_t)(transfer * 1e6), (int64_t)(chunk * 1e6),
                             (int64_t)(tail * 1e6));
  }
  fill_stats(stats, cnt, ms,
             std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - wall0).count());
  return SS_OK;
}

ss_status stream_layers_impl(ss_ctx* ctx, const ss_layers_desc* ld, ss_stream_stats* total) {
  if (!ld || !ld->layers || ld->n_layers <= 0) return SS_ERR_ARG;
  if (ld->mode < SS_LAYERS_PREFETCH || ld->mode > SS_LAYERS_RESTORE) return SS_ERR_ARG;
  if (ld->mode == SS_LAYERS_RESTORE && (!ld->restore_k || ld->restore_tokens <= 0))
    return SS_ERR_ARG;
  if (ld->n_layers > 256) return SS_ERR_SHAPE;
  ss::PipeRes r;
  SS_CK(ss::ctx_pipeline(ctx, &r));
  int n_fills[256];
  for (int l = 0; l < ld->n_layers; ++l) SS_ST(validate_desc(ctx, &ld->layers[l], &n_fills[l]));

  const auto wall0 = std::chrono::steady_clock::now();
  SS_CK(cudaEventRecord(r.ev_t0, r.copy_stream));
  LayerCounts cnt;
  int fill_base = 0;
  const bool restore = ld->mode == SS_LAYERS_RESTORE;
  for (int l = 0; l < ld->n_layers; ++l) {
    if (l > 0 && ld->mode != SS_LAYERS_PREFETCH) {
      // no prefetch: the next layer's copies start only when this layer's work is done
      SS_CK(cudaEventRecord(r.ev_t1, r.attn_stream));
      SS_CK(cudaStreamWaitEvent(r.copy_stream, r.ev_t1, 0));
    }
    SS_ST(enqueue_layer(ctx, &ld->layers[l], r, n_fills[l], restore ? 0 : fill_base,
                        restore ? ld->restore_k : nullptr, restore ? ld->restore_v : nullptr,
                        ld->restore_tokens, &cnt));
    if (!restore) fill_base += n_fills[l];
  }
  SS_CK(cudaEventRecord(r.ev_t1, r.attn_stream));
  SS_CK(cudaEventSynchronize(r.ev_t1));
  SS_CK(cudaStreamSynchronize(r.copy_stream));
  float ms = 0.f;
  SS_CK(cudaEventElapsedTime(&ms, r.ev_t0, r.ev_t1));
  fill_stats(total, cnt, ms,
             std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - wall0).count());
  return SS_OK;
}

}  // namespace

extern "C" ss_status ss_stream_round(ss_ctx* ctx, const ss_stream_desc* d, ss_stream_stats* stats) {
  if (!ctx) return SS_ERR_ARG;
  // a round the caller has open stays as it is: the pipeline only ever drops rounds it opened
  if (ss::ctx_round_open(ctx)) return SS_ERR_STATE;
  ss::ctx_pipeline_mode(ctx, true);
  const ss_status st = stream_round_impl(ctx, d, stats);
  if (st != SS_OK) ss::ctx_pipeline_drain(ctx);
  ss::ctx_pipeline_mode(ctx, false);
  return st;
}

extern "C" ss_status ss_stream_layers(ss_ctx* ctx, const ss_layers_desc* layers, ss_stream_stats* total) {
  if (!ctx) return SS_ERR_ARG;
  if (ss::ctx_round_open(ctx)) return SS_ERR_STATE;
  ss::ctx_pipeline_mode(ctx, true);
  const ss_status st = stream_layers_impl(ctx, layers, total);
  if (st != SS_OK) ss::ctx_pipeline_drain(ctx);
  ss::ctx_pipeline_mode(ctx, false);
  return st;
}
